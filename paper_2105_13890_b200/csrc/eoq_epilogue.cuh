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

// The same rounding on the floating-point pipe, which the integer-heavy epilogue leaves idle.  For an integer t
// with kMagicBits + t inside [2^23, 2^24) the word kMagicBits + t read as a float is 1.5 * 2^23 + t exactly;
// one fused multiply-add forms 1.5 * 2^23 + t / 2^7, whose single rounding (nearest, ties to even, unit spacing
// in that binade) is R(t / 2^7).  Returns kMagicBits + R(t / 2^7): the low 16 bits are the two's-complement code.
constexpr uint32_t kMagicBits = 0x4B400000u;                     // 1.5 * 2^23 as a float
constexpr float kMagicRest = 12582912.0f - 12582912.0f / 128.0f;  // exact: 12484608
__device__ __forceinline__ uint32_t rne7_magic(uint32_t biased)
{
    return __float_as_uint(__fmaf_rn(__uint_as_float(biased), 0.0078125f, kMagicRest));
}

// byte k of w, sign-extended
template <int k>
__device__ __forceinline__ int32_t sbyte(uint32_t w)
{
    // prmt selector digit 8 + k replicates the sign bit of byte k (the __byte_perm intrinsic drops that bit)
    uint32_t r;
    asm("prmt.b32 %0, %1, %1, %2;" : "=r"(r) : "r"(w), "n"(((8 + k) << 12) | ((8 + k) << 8) | ((8 + k) << 4) | k));
    return (int32_t)r;
}

// Forward chain on 16 consecutive output channels of one pixel (Sec. 3.2.1: x2 = Q_a1(conv), x3 = gamma x2,
// x4 = x3 + b2 [+ shortcut], x5 = Q_a2(relu(x4)); mask = [x4 > 0]).  kShift7: the input sits at exponent -7.
// The integer pipe bounds this code, so clamps are moved in front of the roundings (both are monotonic, the
// clamp limits are chosen so that the rounded result is unchanged), roundings run as one FMA each, and the
// constant offsets of that trick are folded into the multiply-add that forms x4.
//
// The b1 term (b1 times the sum of the weights whose taps fall inside the image, per border class and output
// channel) is read from shared memory, already multiplied by b1: the epilogue warps copy the table there once per
// kernel (kTableSmemBytes at most; larger tables are read from global memory and multiplied per use).
constexpr int kTableSmemBytes = 20 * 1024;

// One 256-bit store (sm_100): a whole 32-byte sector per lane instead of two half sectors.  ptr must be 32-byte aligned.
__device__ __forceinline__ void st_global_256(void *ptr, const uint32_t *v)
{
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(ptr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]),
                 "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
                 : "memory");
}

// The three scalar codes of the forward chain as the epilogue uses them: the host values of the launch, or the
// values read from device memory when the caller keeps them there (they then change from one replay of a captured
// graph to the next without a new capture).
struct FwdScalars {
    int32_t b1, gamma, b2;
};

// Every epilogue thread calls this once per kernel.  Device-resident codes outside their range (16 bits each; b1
// also bounded by what keeps the accumulator inside int32) raise EOQ_DEV_RANGE and are clamped.
__device__ __forceinline__ FwdScalars load_fwd_scalars(const IgemmParams &p)
{
    FwdScalars s{p.b1_c, p.gamma_c, p.b2_c};
    if (p.scal_dev) {
        s.b1 = __ldg(p.scal_dev);
        s.gamma = __ldg(p.scal_dev + 1);
        s.b2 = __ldg(p.scal_dev + 2);
        // |acc| <= k_total * (127 + |b1|) * 127 must stay below 2^31 - 2^24
        const long long room = (2147483647ll - 16777216ll) / (127ll * (p.k_total > 0 ? p.k_total : 1)) - 127ll;
        const int32_t b1_lim = (int32_t)(room < 0 ? 0 : (room > 32767 ? 32767 : room));
        const bool bad = s.b1 < -b1_lim || s.b1 > b1_lim || s.gamma < -32768 || s.gamma > 32767 || s.b2 < -32768 ||
                         s.b2 > 32767 || (!p.b1_table && s.b1 != 0);
        if (bad) {
            if (blockIdx.x == 0 && (threadIdx.x & 31) == 0) atomicOr(&p.dev->status, EOQ_DEV_RANGE);
            s.b1 = p.b1_table ? clampi(s.b1, -b1_lim, b1_lim) : 0;
            s.gamma = clampi(s.gamma, -32768, 32767);
            s.b2 = clampi(s.b2, -32768, 32767);
        }
    }
    return s;
}

// Filled by the epilogue warps (`nthreads` of them, `tid` = index among them) before their first tile; they meet at
// named barrier 1 afterwards.  Returns the table's shared-memory address, or null when there is no table or it does
// not fit (uniform over the kernel).
__device__ __forceinline__ const int32_t *stage_b1_table(const IgemmParams &p, int32_t b1, uint8_t *smem_table, int tid, int nthreads)
{
    const int entries = p.b1_table ? p.b1_nrc * p.b1_ncc * p.N : 0;
    if (entries == 0 || entries * (int)sizeof(int32_t) > kTableSmemBytes) return nullptr;
    int32_t *ts = reinterpret_cast<int32_t *>(smem_table);
    for (int i = tid; i < entries; i += nthreads) ts[i] = b1 * __ldg(p.b1_table + i);
    asm volatile("bar.sync 1, %0;" ::"r"(nthreads) : "memory");
    return ts;
}

// `tb`: this pixel's 16 b1 terms in shared memory (already times b1), or null; then `tg` points at the 16 weight
// sums in global memory (or is null when the layer has no b1 term).  `sc`: the 16 shortcut codes (zero without one).
// `acc1` holds the tile's second partial sums when kTwo is set; kRelu = a ReLU follows.
template <bool kShift7, bool kRelu, bool kTwo>
__device__ __forceinline__ void forward_16(const IgemmParams &p, const FwdScalars &fs, const uint32_t (&acc)[32],
                                           const uint32_t (&acc1)[32], size_t off, const int32_t *tb,
                                           const int32_t *tg, const int4 &sc, int shift)
{
    int32_t a[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) a[i] = (int32_t)acc[i];
    bool two = kTwo;
    if (kTwo && (!kShift7 || p.acc_out)) {
        // paths that need the whole sum as a value (the dump, the generic shift) merge the partial sums here;
        // the common path below merges them inside its first clamp
#pragma unroll
        for (int i = 0; i < 16; ++i) a[i] += (int32_t)acc1[i];
        two = false;
    }
    if (tb) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int4 v = reinterpret_cast<const int4 *>(tb)[i];
            a[4 * i + 0] += v.x;
            a[4 * i + 1] += v.y;
            a[4 * i + 2] += v.z;
            a[4 * i + 3] += v.w;
        }
    } else if (tg) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int4 v = __ldg(reinterpret_cast<const int4 *>(tg) + i);
            a[4 * i + 0] += fs.b1 * v.x;
            a[4 * i + 1] += fs.b1 * v.y;
            a[4 * i + 2] += fs.b1 * v.z;
            a[4 * i + 3] += fs.b1 * v.w;
        }
    }
    if (p.acc_out) {
        int4 *d = reinterpret_cast<int4 *>(p.acc_out + off);
#pragma unroll
        for (int i = 0; i < 4; ++i) d[i] = make_int4(a[4 * i], a[4 * i + 1], a[4 * i + 2], a[4 * i + 3]);
    }
    // q = x2 code + q_bias, the code saturated to 16 bits
    uint32_t q[16];
    uint32_t q_bias;
    if (kShift7) {
        // R(a / 2^7) lies in [-32768, 32767] exactly when a lies in [-32768 * 128 - 64, 32767 * 128 + 63], and
        // clamping a to [-32768 * 128, 32767 * 128 + 63] first gives the same code.  |a| < 2^31 - 2^24 (checked
        // on the host), so neither addition below wraps.
        // The lower clamp merges the second partial sum (one add-max); the add of kMagicBits that follows is taken
        // modulo 2^32, where max(A, -2^22) + kMagicBits is the true (positive) sum for every A < 2^31 - 2^24.
        q_bias = kMagicBits;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int32_t lo = two ? __viaddmax_s32(a[i], (int32_t)acc1[i], -4194304) : max(a[i], -4194304);
            q[i] = rne7_magic(__viaddmin_u32((uint32_t)lo, kMagicBits, kMagicBits + 4194239u));
        }
    } else {
        q_bias = 0;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            int32_t v2;
            if (shift >= 0) {
                v2 = rne_shr32(a[i], shift);
            } else {
                const long long w = (long long)a[i] << (-shift);
                v2 = (int32_t)(w < -32768 ? -32768 : (w > 32767 ? 32767 : w));
            }
            q[i] = (uint32_t)clampi(v2, -32768, 32767);
        }
    }
    // x4 - 1 = gamma * x2 + (b2 + shortcut) * 2^7 - 1 = gamma * q + add, the bias of q folded into add (mod 2^32).
    // Forming x4 - 1 instead of x4 makes its sign bit [x4 <= 0], the complement of the mask bit, so the mask
    // costs one funnel shift per element; the + 1 rides on the add-min that clamps x4.
    const uint32_t g = (uint32_t)fs.gamma;
    const uint32_t base = ((uint32_t)fs.b2 << 7) - g * q_bias - 1u;
    uint32_t add[16];
    if (p.shortcut) {
        const int4 v = sc;
        const uint32_t w[4] = {(uint32_t)v.x, (uint32_t)v.y, (uint32_t)v.z, (uint32_t)v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            add[4 * i + 0] = base + (uint32_t)sbyte<0>(w[i]) * 128u;
            add[4 * i + 1] = base + (uint32_t)sbyte<1>(w[i]) * 128u;
            add[4 * i + 2] = base + (uint32_t)sbyte<2>(w[i]) * 128u;
            add[4 * i + 3] = base + (uint32_t)sbyte<3>(w[i]) * 128u;
        }
    } else {
#pragma unroll
        for (int i = 0; i < 16; ++i) add[i] = base;
    }
    // Q_a2: R(x4 / 2^7) saturated to +-127 (and to 0 from below after a ReLU).  16319 / 128 = 127.49.. rounds to
    // 127 and everything above saturates to 127 too, so x4 is clamped to +-16319 before the rounding.
    uint32_t nbits = 0;  // bit i = [x4 <= 0] of channel i
    uint32_t r[16];
#pragma unroll
    for (int i = 15; i >= 0; --i) {
        const int32_t w = (int32_t)(g * q[i] + add[i]);  // x4 - 1
        nbits = __funnelshift_l((uint32_t)w, nbits, 1);
        if (kRelu) r[i] = rne7_magic((uint32_t)__viaddmin_s32_relu(w, 1, 16319) | kMagicBits);
        else r[i] = rne7_magic((uint32_t)max(__viaddmin_s32(w, 1, 16319), -16319) + kMagicBits);
    }
    int4 o;
    o.x = (int)__byte_perm(__byte_perm(r[0], r[1], 0x0040), __byte_perm(r[2], r[3], 0x0040), 0x5410);
    o.y = (int)__byte_perm(__byte_perm(r[4], r[5], 0x0040), __byte_perm(r[6], r[7], 0x0040), 0x5410);
    o.z = (int)__byte_perm(__byte_perm(r[8], r[9], 0x0040), __byte_perm(r[10], r[11], 0x0040), 0x5410);
    o.w = (int)__byte_perm(__byte_perm(r[12], r[13], 0x0040), __byte_perm(r[14], r[15], 0x0040), 0x5410);
    *reinterpret_cast<int4 *>(p.x5 + off) = o;
    if (p.relu_mask) *reinterpret_cast<uint16_t *>(p.relu_mask + (off >> 3)) = (uint16_t)~nbits;
    if (p.x2) {
        uint32_t h[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) h[i] = __byte_perm(q[2 * i], q[2 * i + 1], 0x5410);
        if ((reinterpret_cast<uintptr_t>(p.x2) & 31) == 0) {   // (uniform) the 16 codes of x2 are one 32-byte sector
            st_global_256(p.x2 + off, h);
        } else {
            int4 *d = reinterpret_cast<int4 *>(p.x2 + off);
            d[0] = make_int4((int)h[0], (int)h[1], (int)h[2], (int)h[3]);
            d[1] = make_int4((int)h[4], (int)h[5], (int)h[6], (int)h[7]);
        }
    }
}

// Error back-propagation: keep the exact int32 sums (the scale quantizer needs the maximum over the whole
// tensor before any element can be coded) and track max |.|.
// kWide: the destination is 32-byte aligned (the launch checks the base; off is a multiple of 16 elements)
template <bool kWide>
__device__ __forceinline__ uint32_t dgrad_16(const IgemmParams &p, const uint32_t *acc, size_t off, uint32_t &mx_masked)
{
    uint32_t mx = 0;
    // the consumer's error head needs the maximum over the positions its ReLU lets through as well (off is the element
    // index of the error tensor and a multiple of 16: one 16-bit word of mask bits)
    const uint32_t bits = p.next_mask ? (uint32_t)__ldg(reinterpret_cast<const uint16_t *>(p.next_mask) + (off >> 4)) : 0u;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t a0 = (uint32_t)abs((int)acc[4 * i]), a1 = (uint32_t)abs((int)acc[4 * i + 1]);
        const uint32_t a2 = (uint32_t)abs((int)acc[4 * i + 2]), a3 = (uint32_t)abs((int)acc[4 * i + 3]);
        mx = max(max(mx, a0), max(a1, max(a2, a3)));
        if (bits) {
            const uint32_t b4 = bits >> (4 * i);
            mx_masked = max(mx_masked, (b4 & 1u) ? a0 : 0u);
            mx_masked = max(mx_masked, (b4 & 2u) ? a1 : 0u);
            mx_masked = max(mx_masked, (b4 & 4u) ? a2 : 0u);
            mx_masked = max(mx_masked, (b4 & 8u) ? a3 : 0u);
        }
    }
    if (kWide) {
        st_global_256(p.acc_out + off, acc);
        st_global_256(p.acc_out + off + 8, acc + 8);
    } else {
        int4 *d = reinterpret_cast<int4 *>(p.acc_out + off);
#pragma unroll
        for (int i = 0; i < 4; ++i) d[i] = make_int4((int)acc[4 * i], (int)acc[4 * i + 1], (int)acc[4 * i + 2], (int)acc[4 * i + 3]);
    }
    return mx;
}

}  // namespace eoq
