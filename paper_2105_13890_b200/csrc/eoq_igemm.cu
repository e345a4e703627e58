// Implicit-GEMM convolution kernel for sm_100a: forward pass and error back-propagation of the EOQ layer
// (arXiv 2105.13890, Sec. 3.2.1).  One persistent CTA per SM walks 128-row output tiles:
//   warp 0   : TMA producer (im2col loads of the activation/error operand, tiled loads of the weights)
//   warp 1   : owns tensor memory, issues tcgen05.mma kind::i8 (int8 x int8 -> int32 in TMEM)
//   warps 2-9: epilogue; read the accumulators with tcgen05.ld and apply the layer's quantizers in registers
// Two accumulator buffers in TMEM let the epilogue of tile i overlap the main loop of tile i+1.
// Every wait is bounded: when one runs out the CTA raises EOQ_DEV_TIMEOUT, drains and returns.
#include "eoq_device.cuh"
#include "eoq_internal.h"

namespace eoq {

namespace {

constexpr int kMaxStages = 8;

struct RoleCtx {
    volatile uint32_t *abort_flag;
    DeviceState *dev;
};

__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, const RoleCtx &c)
{
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        if (ptx::mbar_try_wait(bar, parity)) return true;
        if (*c.abort_flag) return false;
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

__global__ void __launch_bounds__(kGemmThreads, 1)
igemm_kernel(const __grid_constant__ IgemmParams p, const __grid_constant__ CUtensorMap map_a,
             const __grid_constant__ CUtensorMap map_b)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[2 * kMaxStages + 5];
    __shared__ uint32_t tmem_base_s;
    __shared__ volatile uint32_t abort_s;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t a_sub = (uint32_t)kTileM * p.kc, b_sub = (uint32_t)p.tile_n * p.kc;
    const uint32_t stage_bytes = (uint32_t)p.subs_per_stage * (a_sub + b_sub);
    const uint32_t bar0 = ptx::smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (kMaxStages + s); };
    auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * kMaxStages + a); };
    auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * kMaxStages + 2 + a); };
    const uint32_t drain_bar = bar0 + 8u * (2 * kMaxStages + 4);

    uint32_t acc_stride = 32;
    while (acc_stride < (uint32_t)p.tile_n) acc_stride <<= 1;
    const uint32_t tmem_cols = 2 * acc_stride;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.num_stages; ++s) {
            ptx::mbar_init(full_bar(s), 1);
            ptx::mbar_init(empty_bar(s), 1);
        }
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(tfull_bar(a), 1);
            ptx::mbar_init(tempty_bar(a), kEpilogueWarps);
        }
        ptx::mbar_init(drain_bar, 1);
        abort_s = 0;
        ptx::fence_barrier_init();
        ptx::prefetch_tensormap(&map_a);
        ptx::prefetch_tensormap(&map_b);
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(&tmem_base_s), tmem_cols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;
    const RoleCtx ctx{&abort_s, p.dev};

    const int num_tiles = p.num_m_tiles * p.num_n_tiles;
    const int k_iters = (p.num_sub + p.subs_per_stage - 1) / p.subs_per_stage;
    const int pix_per_img = p.hq * p.wq;

    if (warp == 0) {
        if (lane == 0) {
            // ------------------------------------------------------------------ TMA producer
            int stage = 0;
            uint32_t phase = 0;
            uint32_t inflight = 0, inflight_parity = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                const int mt = tile / p.num_n_tiles, nt = tile % p.num_n_tiles;
                const int m0 = mt * kTileM;
                const int img = m0 / pix_per_img, rem = m0 % pix_per_img;
                const int cw = (rem % p.wq) * p.src_stride_w + p.base_w;
                const int ch = (rem / p.wq) * p.src_stride + p.base_h;
                for (int kit = 0; kit < k_iters; ++kit) {
                    if (!(ok = wait_bar(empty_bar(stage), phase ^ 1u, ctx))) break;
                    const int s0 = kit * p.subs_per_stage;
                    const int subs = min(p.subs_per_stage, p.num_sub - s0);
                    const uint32_t a_dst = smem_base + stage * stage_bytes;
                    const uint32_t b_dst = a_dst + p.subs_per_stage * a_sub;
                    ptx::mbar_expect_tx(full_bar(stage), subs * (a_sub + b_sub));
                    for (int j = 0; j < subs; ++j) {
                        const int s = s0 + j;
                        const int sd = min(s, p.real_sub - 1);  // a padding sub-tile re-reads real data; its weights are zero
                        const int tap = sd / p.chunks_per_tap, chunk = sd % p.chunks_per_tap;
                        ptx::tma_load_im2col_4d(a_dst + j * a_sub, &map_a, full_bar(stage), chunk * p.kc, cw, ch, img,
                                                (uint16_t)p.tap_dw[tap], (uint16_t)p.tap_dh[tap]);
                        // tap coordinate p.ntaps lies outside the weight tensor: the padding sub-tile is zero-filled
                        ptx::tma_load_3d(b_dst + j * b_sub, &map_b, full_bar(stage), chunk * p.kc,
                                         s < p.real_sub ? (int)p.tap_b[tap] : 0x7fff, nt * p.tile_n);
                    }
                    inflight |= 1u << stage;
                    inflight_parity = (inflight_parity & ~(1u << stage)) | (phase << stage);
                    if (++stage == p.num_stages) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                // wait, bounded, for the copies this thread still has in flight
                for (int s = 0; s < p.num_stages; ++s)
                    if (inflight & (1u << s))
                        for (uint32_t i = 0; i < kSpinLimit; ++i)
                            if (ptx::mbar_try_wait(full_bar(s), (inflight_parity >> s) & 1u)) break;
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ------------------------------------------------------------------ MMA issuer
            const uint32_t idesc = make_idesc_i8(kTileM, p.tile_n, false, false);
            const uint32_t lt = layout_type_for(p.kc);
            int stage = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                if (!(ok = wait_bar(tempty_bar(acc), acc_phase ^ 1u, ctx))) break;
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * acc_stride;
                uint32_t accumulate = 0;
                for (int kit = 0; kit < k_iters; ++kit) {
                    if (!(ok = wait_bar(full_bar(stage), phase, ctx))) break;
                    ptx::tc_fence_after();
                    const int subs = min(p.subs_per_stage, p.num_sub - kit * p.subs_per_stage);
                    const uint32_t a_base = smem_base + stage * stage_bytes;
                    const uint32_t b_base = a_base + p.subs_per_stage * a_sub;
                    if (p.kc >= 32) {
                        // swizzled K-major sub-tiles: rows kc bytes wide, 8-row groups 8*kc apart; a 32-byte
                        // K step moves the start address inside the swizzle span
                        const uint32_t sbo = 8u * p.kc;
                        for (int j = 0; j < subs; ++j)
                            for (int kk = 0; kk < p.kc; kk += 32) {
                                ptx::mma_i8(d_tmem, make_smem_desc(a_base + j * a_sub + kk, 0, sbo, lt),
                                            make_smem_desc(b_base + j * b_sub + kk, 0, sbo, lt), idesc, accumulate);
                                accumulate = 1;
                            }
                    } else {
                        // 16-byte rows, no swizzle: one MMA spans two sub-tiles (two taps); the second half of
                        // K sits one sub-tile further (leading offset), 8-row groups are 128 bytes apart
                        for (int j = 0; j < subs; j += 2) {
                            ptx::mma_i8(d_tmem, make_smem_desc(a_base + j * a_sub, a_sub, 128, 0),
                                        make_smem_desc(b_base + j * b_sub, b_sub, 128, 0), idesc, accumulate);
                            accumulate = 1;
                        }
                    }
                    ptx::mma_commit(empty_bar(stage));
                    if (++stage == p.num_stages) { stage = 0; phase ^= 1u; }
                }
                if (ok) ptx::mma_commit(tfull_bar(acc));
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
            if (!ok) {
                ptx::mma_commit(drain_bar);
                for (uint32_t i = 0; i < kSpinLimit; ++i)
                    if (ptx::mbar_try_wait(drain_bar, 0)) break;
            }
        }
    } else {
        // ---------------------------------------------------------------------- epilogue
        // Eight warps, two per scheduler: a warp may read the TMEM lanes of quadrant (warp % 4); the two warps
        // of a quadrant split the tile's columns.
        const int quad = warp & 3;
        const int half = (warp - 2) >> 2;
        const int row = quad * 32 + lane;
        const int groups = p.tile_n / 16;                 // 16-column groups of the tile
        const int g_begin = half ? (groups + 1) / 2 : 0;  // the first half takes the odd group
        const int g_end = half ? groups : (groups + 1) / 2;
        int shift = 7;
        if (p.epilogue == kEpiForward && p.x_exp) {
            shift = -__ldg(p.x_exp);
            if (shift > 31 || shift < -16) {
                if (lane == 0) atomicOr(&p.dev->status, EOQ_DEV_RANGE);
                shift = max(-16, min(31, shift));
            }
        }
        int acc = 0;
        uint32_t acc_phase = 0, mx = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
            const int mt = tile / p.num_n_tiles, nt = tile % p.num_n_tiles;
            if (!(ok = __all_sync(0xffffffffu, wait_bar(tfull_bar(acc), acc_phase, ctx)))) break;  // warp-uniform
            ptx::tc_fence_after();
            const int m = mt * kTileM + row;
            const bool valid = m < p.M;
            size_t pix = 0;
            int cls = 0;
            if (valid) {
                const int img = m / pix_per_img, rem = m % pix_per_img;
                const int y = rem / p.wq, x = rem % p.wq;
                pix = ((size_t)img * p.out_h + (y * p.out_step + p.out_off_h)) * p.out_w + (x * p.out_step + p.out_off_w);
                if (p.b1_table)
                    cls = border_class(y, p.hq, p.b1_nlo_h, p.b1_nhi_h, p.b1_nrc) * p.b1_ncc +
                          border_class(x, p.wq, p.b1_nlo_w, p.b1_nhi_w, p.b1_ncc);
            }
            const uint32_t t_row = tmem_base + acc * acc_stride + ((uint32_t)(quad * 32) << 16);
            for (int g = g_begin; g < g_end; ++g) {
                uint32_t r[32];
                ptx::tmem_ld_32x16(t_row + g * 16, r);
                ptx::tmem_ld_wait();
                const int col = nt * p.tile_n + g * 16;
                if (valid && col < p.N) {
                    const size_t off = pix * p.N + col;
                    if (p.epilogue == kEpiForward) {
                        if (shift == 7) forward_16<true>(p, r, off, col, cls, shift);
                        else forward_16<false>(p, r, off, col, cls, shift);
                    } else {
                        mx = max(mx, dgrad_16(p, r, off));
                    }
                }
            }
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(tempty_bar(acc));
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
        if (p.epilogue == kEpiDgrad) {
            mx = warp_max_u32(mx);
            if (lane == 0 && mx) atomicMax(&p.dev->absmax_u32, mx);
        }
    }

    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, tmem_cols);
    }
}

}  // namespace

size_t igemm_smem_bytes(const IgemmParams &p)
{
    return (size_t)p.num_stages * p.subs_per_stage * ((size_t)kTileM + p.tile_n) * p.kc + 1024;
}

cudaError_t launch_igemm(const IgemmParams &p, const CUtensorMap &map_a, const CUtensorMap &map_b, int grid,
                         cudaStream_t stream)
{
    const size_t smem = igemm_smem_bytes(p);
    cudaError_t e = cudaFuncSetAttribute(igemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 208 * 1024);
    if (e != cudaSuccess) return e;
    igemm_kernel<<<grid, kGemmThreads, smem, stream>>>(p, map_a, map_b);
    return cudaGetLastError();
}

}  // namespace eoq
