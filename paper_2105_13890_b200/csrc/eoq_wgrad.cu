// Weight-gradient kernel for sm_100a (arXiv 2105.13890, Sec. 3.2.1: g_w = Q_g(e3 * x1)).
//   D[(tap, ic), oc] = sum over error pixels q of  x[q shifted by tap, ic] * e3[q, oc]
// The reduction runs over pixels, which is the slow axis of both NHWC operands, so both are fed to
// tcgen05.mma as MN-major tiles: a TMA im2col load brings [pixels][channels] of the activation for one
// filter tap, a tiled TMA load brings [pixels][channels] of the error.  The pixel range is split across
// CTAs (split-K); int32 partial sums leave TMEM and are combined exactly with 64-bit atomics.
// Roles: warps 0, 2, 3 TMA producers (a thread gets a TMA instruction out only every few hundred cycles, threads
// of different warps issue side by side: the loads of every stage are dealt out over three producers), warp 1
// MMA issuer and TMEM owner, warps 4-7 epilogue.  All waits are bounded.
#include "eoq_device.cuh"
#include "eoq_internal.h"

namespace eoq {

namespace {

constexpr int kMaxStages = 8;
constexpr int kProducers = 3;

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

// Descriptor of an MN-major operand made of sub-tiles [pixels][row_bytes], `sub_bytes` apart along M/N.
// Swizzled rows: atoms along M/N are `sub_bytes` apart (leading offset), 8-pixel groups 8*row_bytes apart
// (stride offset).  16-byte rows carry no swizzle and the two offsets swap roles.
__device__ __forceinline__ uint64_t mn_major_desc(uint32_t addr, int row_bytes, uint32_t sub_bytes)
{
    if (row_bytes == 16) return make_smem_desc(addr, 128, sub_bytes, 0);
    return make_smem_desc(addr, sub_bytes, 8u * row_bytes, layout_type_for(row_bytes));
}

__global__ void __launch_bounds__(kWgradThreads, 1)
wgrad_kernel(const __grid_constant__ WgradParams p, const __grid_constant__ CUtensorMap map_x,
             const __grid_constant__ CUtensorMap map_e)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[2 * kMaxStages + 2];
    __shared__ uint32_t tmem_base_s;
    __shared__ volatile uint32_t abort_s;

    const int warp = warp_index_uniform(), lane = threadIdx.x & 31;
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    const int px = p.pixels_per_stage;
    const uint32_t a_sub = (uint32_t)px * p.kc, b_sub = (uint32_t)px * p.nc;
    const int b_subs = p.tile_n / p.nc;
    const uint32_t a_mtile = (uint32_t)p.subs_per_mtile * a_sub;  // bytes of one M tile's activation sub-tiles
    const uint32_t stage_bytes = (uint32_t)p.mtiles_per_cta * a_mtile + (uint32_t)b_subs * b_sub;
    const uint32_t bar0 = ptx::smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (kMaxStages + s); };
    const uint32_t done_bar = bar0 + 8u * (2 * kMaxStages);

    uint32_t tmem_cols = 32;
    while (tmem_cols < (uint32_t)(p.mtiles_per_cta * p.tile_n)) tmem_cols <<= 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.num_stages; ++s) {
            ptx::mbar_init(full_bar(s), kProducers);  // every producer announces its share of the stage's bytes
            ptx::mbar_init(empty_bar(s), 1);
        }
        ptx::mbar_init(done_bar, 1);
        abort_s = 0;
        ptx::fence_barrier_init();
        ptx::prefetch_tensormap(&map_x);
        ptx::prefetch_tensormap(&map_e);
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

    // work unit of this CTA
    const int tiles = p.num_m_groups * p.num_n_tiles;
    const int ks = blockIdx.x / tiles, tile = blockIdx.x % tiles;
    const int mt0 = (tile / p.num_n_tiles) * p.mtiles_per_cta, nt = tile % p.num_n_tiles;
    const int my_mtiles = min(p.mtiles_per_cta, p.num_m_tiles - mt0);  // M tiles this CTA accumulates
    const int total_subs = p.ntaps * p.chunks_per_tap;
    int subs_total = 0;  // activation sub-tiles this CTA loads per stage
    for (int jm = 0; jm < my_mtiles; ++jm) subs_total += min(p.subs_per_mtile, total_subs - (mt0 + jm) * p.subs_per_mtile);
    const int q_begin = ks * p.stages_per_split * px;
    int my_stages = p.stages_per_split;
    {
        const int remaining = (p.P - q_begin + px - 1) / px;
        my_stages = remaining < my_stages ? remaining : my_stages;
        if (my_stages < 0) my_stages = 0;
    }

    if (warp == 0 || warp == 2 || warp == 3) {
        if (lane == 0) {
            // producer q issues the loads number q, q + 3, q + 6, ... of every stage (activation sub-tiles first,
            // then the error sub-tiles)
            const int q = warp == 0 ? 0 : warp - 1;
            const int n_ops = subs_total + b_subs;
            uint32_t my_bytes = 0;
            for (int o = q; o < n_ops; o += kProducers) my_bytes += o < subs_total ? a_sub : b_sub;
            int stage = 0;
            uint32_t phase = 0, inflight = 0, inflight_parity = 0;
            bool ok = true;
            const int pix_per_img = p.ho * p.wo;
            for (int it = 0; it < my_stages; ++it) {
                if (!(ok = wait_bar(empty_bar(stage), phase ^ 1u, ctx))) break;
                const int q0 = q_begin + it * px;
                const int img = q0 / pix_per_img, rem = q0 % pix_per_img;
                const int cw = (rem % p.wo) * p.src_stride_w + p.base_w;
                const int ch = (rem / p.wo) * p.src_stride + p.base_h;
                const uint32_t a_dst = smem_base + stage * stage_bytes;
                const uint32_t b_dst = a_dst + p.mtiles_per_cta * a_mtile;
                ptx::mbar_expect_tx(full_bar(stage), my_bytes);
                int o = 0;
                for (int jm = 0; jm < my_mtiles; ++jm) {
                    const int first_sub = (mt0 + jm) * p.subs_per_mtile;
                    const int subs = min(p.subs_per_mtile, total_subs - first_sub);  // sub-tiles of this M tile that exist
                    for (int j = 0; j < subs; ++j, ++o) {
                        if (o % kProducers != q) continue;
                        const int s = first_sub + j;
                        const int tap = s / p.chunks_per_tap, chunk = s % p.chunks_per_tap;
                        ptx::tma_load_im2col_4d(a_dst + jm * a_mtile + j * a_sub, &map_x, full_bar(stage), chunk * p.kc, cw, ch,
                                                img, (uint16_t)p.tap_dw[tap], (uint16_t)p.tap_dh[tap]);
                    }
                }
                for (int j = 0; j < b_subs; ++j, ++o)
                    if (o % kProducers == q)
                        ptx::tma_load_2d(b_dst + j * b_sub, &map_e, full_bar(stage), nt * p.tile_n + j * p.nc, q0);
                inflight |= 1u << stage;
                inflight_parity = (inflight_parity & ~(1u << stage)) | (phase << stage);
                if (++stage == p.num_stages) { stage = 0; phase ^= 1u; }
            }
            if (!ok) {
                for (int s = 0; s < p.num_stages; ++s)
                    if (inflight & (1u << s))
                        for (uint32_t i = 0; i < kSpinLimit; ++i)
                            if (ptx::mbar_try_wait(full_bar(s), (inflight_parity >> s) & 1u)) break;
            }
        }
    } else if (warp == 1) {
        // the whole warp runs the issue loop; one elected lane issues the MMAs and commits (see elect_one)
        const uint32_t leader = elect_one();
        const uint32_t tmem_base = __shfl_sync(0xffffffffu, tmem_base_s, 0);
        const uint32_t idesc = make_idesc_i8(kTileM, p.tile_n, true, true);
        // descriptor halves that do not change; the loop adds row offsets to the low halves
        const uint64_t a_proto = mn_major_desc(0, p.kc, a_sub), b_proto = mn_major_desc(0, p.nc, b_sub);
        const uint32_t a_hi = (uint32_t)(a_proto >> 32), b_hi = (uint32_t)(b_proto >> 32);
        const uint32_t a_lead = (uint32_t)a_proto, b_lead = (uint32_t)b_proto;  // leading-offset field, address 0
        const uint32_t a_step16 = (32u * p.kc) >> 4, b_step16 = (32u * p.nc) >> 4;  // 32 pixels further down
        const uint32_t a_mtile16 = a_mtile >> 4;
        int stage = 0;
        uint32_t phase = 0, accumulate = 0;
        bool ok = true;
        for (int it = 0; it < my_stages; ++it) {
            if (!(ok = __all_sync(0xffffffffu, wait_bar(full_bar(stage), phase, ctx)))) break;
            ptx::tc_fence_after();
            uint32_t a_lo = ((smem_base + stage * stage_bytes) >> 4) | a_lead;
            uint32_t b_lo = (((smem_base + stage * stage_bytes) >> 4) + ((p.mtiles_per_cta * a_mtile) >> 4)) | b_lead;
            for (int k = 0; k < px; k += 32) {
                // the M tiles of the group meet the same error tile; each has its own accumulator columns
                uint32_t a_j = a_lo, d_j = tmem_base;
                for (int jm = 0; jm < my_mtiles; ++jm, a_j += a_mtile16, d_j += p.tile_n)
                    ptx::mma_i8(d_j, smem_desc_join(a_j, a_hi), smem_desc_join(b_lo, b_hi), idesc, accumulate, leader);
                accumulate = 1;
                a_lo += a_step16;
                b_lo += b_step16;
            }
            ptx::mma_commit(empty_bar(stage), leader);
            if (++stage == p.num_stages) { stage = 0; phase ^= 1u; }
        }
        ptx::mma_commit(done_bar, leader);
        if (!ok)
            for (uint32_t i = 0; i < kSpinLimit; ++i)
                if (ptx::mbar_try_wait(done_bar, 0)) break;
    } else {
        const int quad = warp & 3;
        bool ok = __all_sync(0xffffffffu, wait_bar(done_bar, 0, ctx));
        if (ok && my_stages > 0) ptx::tc_fence_after();
        for (int jm = 0; jm < my_mtiles && ok && my_stages > 0; ++jm) {
            const int mt = mt0 + jm;
            int row = mt * kTileM + quad * 32 + lane;  // (tap, ic) flattened: tap * c_in + ic
            bool valid = row < p.rows_total;
            if (p.row_window_kw) {
                // filter-row path: the rows are (filter row, tap 0..7, channel): drop the padding taps
                const int per_frow = 8 * p.c_in, fr = row / per_frow, within = row % per_frow;
                const int t = within / p.c_in;
                valid = fr < p.ntaps && t < p.row_window_kw;
                row = (fr * p.row_window_kw + t) * p.c_in + within % p.c_in;
            }
            const uint32_t t_row = tmem_base + jm * p.tile_n + ((uint32_t)(quad * 32) << 16);
            for (int c0 = 0; c0 < p.tile_n; c0 += 32) {
                uint32_t r[32];
                const int ncol = min(32, p.tile_n - c0);
                if (ncol == 32) ptx::tmem_ld_32x32(t_row + c0, r);
                else ptx::tmem_ld_32x16(t_row + c0, r);
                ptx::tmem_ld_wait();
                if (valid) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const int oc = nt * p.tile_n + c0 + j;
                        if (j < ncol && oc < p.c_out) {
                            const long long v = (int32_t)r[j];
                            if (v) atomicAdd(reinterpret_cast<unsigned long long *>(p.acc + (size_t)oc * p.rows_total + row),
                                             (unsigned long long)v);
                        }
                    }
                }
            }
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

size_t wgrad_smem_bytes(const WgradParams &p)
{
    const size_t stage = (size_t)p.mtiles_per_cta * p.subs_per_mtile * p.pixels_per_stage * p.kc +
                         (size_t)p.tile_n * p.pixels_per_stage;
    return stage * p.num_stages + 1024;
}

cudaError_t launch_wgrad(const WgradParams &p, const CUtensorMap &map_x, const CUtensorMap &map_e, cudaStream_t stream)
{
    cudaError_t e = cudaFuncSetAttribute(wgrad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 208 * 1024);
    if (e != cudaSuccess) return e;
    const int grid = p.num_m_groups * p.num_n_tiles * p.num_k_splits;
    wgrad_kernel<<<grid, kWgradThreads, wgrad_smem_bytes(p), stream>>>(p, map_x, map_e);
    return cudaGetLastError();
}

}  // namespace eoq
