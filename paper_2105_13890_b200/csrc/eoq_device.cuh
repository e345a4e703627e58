// Device-side helpers: integer rounding of the EOQ quantizers and thin wrappers over sm_100a PTX.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace eoq {

// ------------------------------------------------------------------ integer rounding (Sec. 3.2.2)

// R(a / 2^s), nearest with ties to even, for s in [0, 31].
__device__ __forceinline__ int32_t rne_shr32(int32_t a, int s)
{
    if (s == 0) return a;
    int32_t q = a >> s;
    uint32_t r = (uint32_t)a & ((1u << s) - 1u);
    uint32_t h = 1u << (s - 1);
    return q + (int32_t)((r > h) || (r == h && (q & 1)));
}

// R(a / 2^s) for 64-bit a and s in [0, 62].
__device__ __forceinline__ long long rne_shr64(long long a, int s)
{
    if (s == 0) return a;
    long long q = a >> s;
    unsigned long long r = (unsigned long long)a & ((1ull << s) - 1ull);
    unsigned long long h = 1ull << (s - 1);
    return q + (long long)((r > h) || (r == h && (q & 1)));
}

__device__ __forceinline__ int32_t clampi(int32_t v, int32_t lo, int32_t hi) { return min(max(v, lo), hi); }

// R(log2 M) for M >= 1: floor(log2 M) plus one when M^2 >= 2^(2f+1).
__device__ __forceinline__ int round_log2_u32(uint32_t M)
{
    int f = 31 - __clz(M);
    unsigned long long sq = (unsigned long long)M * M;
    return f + (sq >= (1ull << (2 * f + 1)) ? 1 : 0);
}

__device__ __forceinline__ int round_log2_u64(unsigned long long M)
{
    if (M < (1ull << 32)) return round_log2_u32((uint32_t)M);
    int f = 63 - __clzll(M);
    unsigned long long hi = __umul64hi(M, M);  // M^2 >= 2^(2f+1) with 2f+1 >= 65
    return f + (hi >= (1ull << (2 * f + 1 - 64)) ? 1 : 0);
}

// Code of SQ for an integer a once t = R(log2 max) is known: sat(R(a * 2^(7-t)), -127, 127).
__device__ __forceinline__ int32_t sq_code32(int32_t a, int t)
{
    int s = t - 7;
    int32_t v = s >= 0 ? rne_shr32(a, s) : a * (1 << (-s));  // s < 0 only when |a| < 2^7.5
    return clampi(v, -127, 127);
}

// The same code for a shift s = t - 7 >= 1 known to the whole kernel, in four integer operations before the
// clamp: adding 2^(s-1) - 1 plus the parity of the quotient carries into bit s exactly when the remainder exceeds
// one half, or equals it with an odd quotient.  `half_m1` = 2^(s-1) - 1.  Needs |a| + 2^(s-1) < 2^31, which holds
// because 2^(s-1) <= max|a| / 2^7.
__device__ __forceinline__ int32_t sq_code32_shr(int32_t a, int s, int32_t half_m1)
{
    return clampi((a + half_m1 + ((a >> s) & 1)) >> s, -127, 127);
}

__device__ __forceinline__ int32_t sq_code64(long long a, int t)
{
    int s = t - 7;
    long long v = s >= 0 ? rne_shr64(a, s) : a * (1ll << (-s));
    return (int32_t)(v < -127 ? -127 : (v > 127 ? 127 : v));
}

// ------------------------------------------------------------------ border classes of the b1 term
// x1 = x0 + b1 has a zero halo, so conv(x1) = conv(x0) + b1 * (sum of the weights of the taps that fall
// inside the image).  Which taps are inside depends only on how far the output row (column) is from the
// image border: rows whose window sticks out at the top (y < nlo) or at the bottom (y >= extent - nhi) get a
// class each, all interior rows share class nlo.  When the image is so small that no interior row exists
// (ncls == extent) every row is its own class.

__device__ __forceinline__ int border_class(int y, int extent, int nlo, int nhi, int ncls)
{
    if (ncls == extent) return y;
    if (y < nlo) return y;
    if (y >= extent - nhi) return nlo + 1 + (y - (extent - nhi));
    return nlo;
}

// Is filter tap k inside the image for the rows of class `cls`?
__device__ __forceinline__ bool tap_valid(int cls, int k, int extent_out, int extent_in, int nlo, int nhi, int ncls,
                                          int stride, int pad)
{
    int y;
    if (ncls == extent_out) y = cls;
    else if (cls < nlo) y = cls;
    else if (cls == nlo) y = nlo;
    else y = extent_out - nhi + (cls - nlo - 1);
    const int src = y * stride - pad + k;
    return src >= 0 && src < extent_in;
}

// ------------------------------------------------------------------ warp reductions

__device__ __forceinline__ uint32_t warp_max_u32(uint32_t v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = max(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

__device__ __forceinline__ long long warp_sum_i64(long long v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Block-wide reductions (every thread of the block must call; the result is valid in thread 0).  Thousands of
// warps hitting one global cell with an atomic serialise at the L2, so each block sends one.
__device__ __forceinline__ unsigned long long block_max_u64(unsigned long long v)
{
    __shared__ unsigned long long red_max[32];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long other = __shfl_xor_sync(0xffffffffu, v, o);
        v = other > v ? other : v;
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = (blockDim.x + 31) >> 5;
    if (lane == 0) red_max[warp] = v;
    __syncthreads();
    if (warp == 0) {
        v = lane < nw ? red_max[lane] : 0ull;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const unsigned long long other = __shfl_xor_sync(0xffffffffu, v, o);
            v = other > v ? other : v;
        }
    }
    __syncthreads();
    return v;
}

__device__ __forceinline__ long long block_sum_i64(long long v)
{
    __shared__ long long red_sum[32];
    v = warp_sum_i64(v);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = (blockDim.x + 31) >> 5;
    if (lane == 0) red_sum[warp] = v;
    __syncthreads();
    if (warp == 0) v = warp_sum_i64(lane < nw ? red_sum[lane] : 0ll);
    __syncthreads();
    return v;
}

// ------------------------------------------------------------------ PTX: shared-memory barriers and TMA

namespace ptx {

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_barrier_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Tiled TMA loads (global -> shared), completion counted in bytes on an mbarrier.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const void *map, uint32_t bar, int c0, int c1)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const void *map, uint32_t bar, int c0, int c1, int c2)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const void *map, uint32_t bar, int c0, int c1, int c2, int c3)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}
// im2col-mode TMA load on a rank-4 (C, W, H, N) tensor: coordinates of the first pixel plus the
// filter-tap offsets (w, h).
__device__ __forceinline__ void tma_load_im2col_4d(uint32_t dst, const void *map, uint32_t bar, int c, int w, int h,
                                                   int n, uint16_t off_w, uint16_t off_h)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%3, %4, %5, %6}], [%2], {%7, %8};"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n), "h"(off_w), "h"(off_h)
        : "memory");
}
__device__ __forceinline__ void prefetch_tensormap(const void *map)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

// ------------------------------------------------------------------ PTX: tensor memory and tcgen05

__device__ __forceinline__ void tmem_alloc(uint32_t smem_result, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_result), "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// The warp that feeds the tensor core runs its whole loop with all 32 lanes (so that every address and
// descriptor it computes is the same in all lanes and can live in the uniform datapath, which is where the MMA
// instruction takes its operands from) and only the instructions that must come from a single thread are
// predicated on one elected lane.  Issued from inside a one-lane branch instead, every operand has to be moved
// from a vector to a uniform register per MMA, which costs more cycles than a narrow MMA takes.

// 1 in exactly one lane of the (fully active) warp, 0 in the others.
__device__ __forceinline__ uint32_t elect_one()
{
    uint32_t leader;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "elect.sync _|p, 0xffffffff;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(leader));
    return leader;
}

// Index of the calling warp in its block, in a form the compiler knows to be the same in all lanes.
__device__ __forceinline__ int warp_index_uniform() { return __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0); }

// D[tmem] (+)= A[smem desc] * B[smem desc], int8 x int8 -> int32, issued by the lane whose `leader` is non-zero.
// (No memory clobber: the issuing warp's scalar work between two MMAs is what limits narrow tiles, so the
// compiler must be free to keep loop state in registers.  Ordering against barrier waits and commits comes from
// those being volatile asm statements with memory clobbers.)
__device__ __forceinline__ void mma_i8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate, uint32_t leader)
{
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "setp.ne.b32 q, %5, 0;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(leader));
}

// The mbarrier receives one arrival when every MMA issued so far by the leader lane has completed.
__device__ __forceinline__ void mma_commit(uint32_t bar, uint32_t leader)
{
    asm volatile(
        "{\n\t.reg .pred q;\n\t"
        "setp.ne.b32 q, %1, 0;\n\t"
        "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
        ::"r"(bar), "r"(leader) : "memory");
}

// 32 lanes x 32 columns of 32-bit accumulators: thread t of the warp receives lane (base lane + t).
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_32x16(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

}  // namespace ptx

using ptx::elect_one;
using ptx::warp_index_uniform;

// 64-bit shared-memory matrix descriptor of tcgen05.mma (start address, leading and stride byte offsets
// in 16-byte units, descriptor version 1 at bit 46, swizzle mode at bits 61..63).
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes,
                                                   uint32_t layout_type)
{
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | ((uint64_t)layout_type << 61);
}

// The same descriptor split in two 32-bit halves, so that an issue loop only adds byte offsets (in 16-byte
// units) to the low half: low = start address >> 4 | (leading offset >> 4) << 16, high = (stride offset >> 4) |
// version bit | swizzle mode.  Building the whole descriptor per MMA costs more cycles than a narrow MMA takes.
__device__ __forceinline__ uint32_t smem_desc_hi(uint32_t sbo_bytes, uint32_t layout_type)
{
    return ((sbo_bytes >> 4) & 0x3FFFu) | (1u << 14) | (layout_type << 29);
}
__device__ __forceinline__ uint64_t smem_desc_join(uint32_t lo, uint32_t hi) { return ((uint64_t)hi << 32) | lo; }

// The warp that feeds the tensor core is a single in-order instruction stream: about 25 scalar instructions
// per MMA cost ~130 cycles, while a 128 x 64 x 32 MMA takes 52.  The issue helpers below are therefore fully
// unrolled with compile-time MMA indices, so that an MMA costs a handful of integer adds.
//
// Successive MMAs of a tile alternate between two partial accumulators d0 / d1 when the tile has them (an MMA
// that accumulates into the columns its predecessor is still writing waits ~97 cycles; two interleaved chains
// run at 52 cycles for 64 columns, 69 for 128).  `fresh` is 1 for the first MMAs of a tile, which overwrite.

// kSteps 32-byte K steps of one (A sub-tile, B sub-tile) pair; `parity` = index of the first MMA modulo 2.
// The B operand has its own descriptor half `b_hi` and its own K step `b_k16` (16-byte units): 2 for a K-major
// tile (32 bytes along the row), 2 * row bytes for an MN-major one (32 rows further).
template <int kSteps>
__device__ __forceinline__ void mma_k_steps(uint32_t d0, uint32_t d1, uint32_t a_lo, uint32_t b_lo, uint32_t hi,
                                            uint32_t idesc, uint32_t parity, uint32_t fresh0, uint32_t fresh1,
                                            uint32_t leader, uint32_t b_hi, uint32_t b_k16)
{
#pragma unroll
    for (int kk = 0; kk < kSteps; ++kk) {
        const bool odd = ((kk & 1) != 0) != (parity != 0);
        // the first MMA into each accumulator overwrites it
        uint32_t acc = 1u;
        if (kk < 2) acc = (odd ? fresh1 : fresh0) ? 0u : 1u;
        ptx::mma_i8(odd ? d1 : d0, smem_desc_join(a_lo + 2 * kk, hi), smem_desc_join(b_lo + kk * b_k16, b_hi), idesc, acc, leader);
    }
}

// All kDim x kDim taps of one channel chunk against resident weights: tap (a, b) reads the patch tile
// (a * row16 + b * kc16) further (16-byte units); its weights are the next sub-tile.
template <int kDim, int kSteps>
__device__ __forceinline__ void mma_patch_chunk(uint32_t d0, uint32_t d1, uint32_t a_lo, uint32_t b_lo, uint32_t row16,
                                                uint32_t kc16, uint32_t b_sub16, uint32_t hi, uint32_t idesc,
                                                bool first_chunk, bool two_acc, uint32_t leader, uint32_t b_hi,
                                                uint32_t b_k16)
{
#pragma unroll
    for (int a = 0; a < kDim; ++a)
#pragma unroll
        for (int b = 0; b < kDim; ++b)
#pragma unroll
            for (int kk = 0; kk < kSteps; ++kk) {
                const int idx = (a * kDim + b) * kSteps + kk;
                uint32_t acc = 1u;
                if (idx == 0) acc = first_chunk ? 0u : 1u;
                if (idx == 1) acc = (first_chunk && two_acc) ? 0u : 1u;
                ptx::mma_i8((idx & 1) ? d1 : d0, smem_desc_join(a_lo + a * row16 + b * kc16 + 2 * kk, hi),
                            smem_desc_join(b_lo + (a * kDim + b) * b_sub16 + kk * b_k16, b_hi), idesc, acc, leader);
            }
}
// Swizzle field of the descriptor for a sub-tile whose rows are `row_bytes` wide.
__device__ __forceinline__ uint32_t layout_type_for(int row_bytes)
{
    return row_bytes == 128 ? 2u : (row_bytes == 64 ? 4u : (row_bytes == 32 ? 6u : 0u));
}

// 32-bit instruction descriptor of tcgen05.mma kind::i8: signed 8-bit A and B, int32 accumulator, M x N.
__device__ __forceinline__ uint32_t make_idesc_i8(int m, int n, bool a_mn_major, bool b_mn_major)
{
    return (2u << 4) | (1u << 7) | (1u << 10) | ((a_mn_major ? 1u : 0u) << 15) | ((b_mn_major ? 1u : 0u) << 16) |
           ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

}  // namespace eoq
