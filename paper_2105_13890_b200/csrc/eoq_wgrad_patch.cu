// Patch variant of the weight-gradient kernel for stride-1 filters (arXiv 2105.13890, Sec. 3.2.1:
// g_w = Q_g(e3 * x1)):  G[oc, (a, b), ic] = sum over error pixels (n, y, x) of e3[n, y, x, oc] * x[n, y + a - p, x + b - p, ic].
//
// The TMA engine delivers a row every ~4.7 cycles, so loading the activation once per tap (9 rows per pixel for a
// 3x3 filter) starves the tensor core.  Here the reduction axis is the raster of a pixel block: r_rows output rows
// of one image, each widened to pw = wo + k - 1 pixels.  The error patch is loaded with zeros in the extra columns
// (TMA out-of-bounds fill); the activation patch carries k - 1 more rows and starts p pixels up and left.  In that
// raster the activation pixel that meets error pixel r under tap (a, b) is pixel r + a * pw + b, so every tap is the
// same shared-memory tile read through a descriptor started that many rows further (MN-major operands, the swizzle
// is a function of the address).  One row per pixel is loaded for the activation and one for the error whatever
// the filter size.
//
// An accumulator holds 128 / kc horizontally adjacent taps of one filter row (M = 128 rows = taps x channels of the
// chunk; the atoms of the MN-major operand are one pixel apart).  A CTA owns the accumulators of a few filter rows
// for one input-channel chunk and one output-channel tile, runs them over a range of pixel blocks, and stores int32
// partial sums in its own slice; a finishing kernel adds the slices in 64 bits.
// Roles: warp 0 TMA loads, warp 1 TMEM owner + MMA issuer, warps 2-5 epilogue.  All waits are bounded.
#include "eoq_device.cuh"
#include "eoq_epilogue.cuh"
#include "eoq_internal.h"

namespace eoq {

namespace {

constexpr int kMaxStages = 4;
constexpr int kMaxAcc = 8;

__global__ void __launch_bounds__(kWgradPatchThreads, 1)
wgrad_patch_kernel(const __grid_constant__ WgradPatchPlan pl, const __grid_constant__ CUtensorMap map_x,
                   const __grid_constant__ CUtensorMap map_e)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[2 * kMaxStages + 1];
    __shared__ uint32_t tmem_base_s;
    __shared__ volatile uint32_t abort_s;

    const int warp = warp_index_uniform(), lane = threadIdx.x & 31;
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t stage_bytes = (uint32_t)(pl.x_bytes + pl.e_bytes);
    const uint32_t bar0 = ptx::smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (kMaxStages + s); };
    const uint32_t done_bar = bar0 + 8u * (2 * kMaxStages);

    // this CTA's group and range of pixel blocks
    const int g = blockIdx.x % pl.num_groups, ks = blockIdx.x / pl.num_groups;
    const int rg = g % pl.row_groups, c = (g / pl.row_groups) % pl.chunks, nt = g / (pl.row_groups * pl.chunks);
    const int row0 = rg * pl.rows_per_group;
    const int rows_here = min(pl.rows_per_group, pl.kdim - row0);
    const int num_acc = rows_here * pl.accs_per_row;
    const int total_blocks = pl.n_img * pl.blocks_per_img;
    const int blk_begin = ks * pl.blocks_per_split;
    const int blk_end = min(total_blocks, blk_begin + pl.blocks_per_split);
    const int my_blocks = max(0, blk_end - blk_begin);

    uint32_t tmem_cols = 32;
    while (tmem_cols < (uint32_t)(num_acc * pl.tile_n)) tmem_cols <<= 1;

    // The error buffers' rows between r_rows * pw and kp are never written by a load: clear them once, so that the
    // rounded-up tail of the reduction adds nothing.
    {
        const int tail_bytes = (pl.kp - pl.r_rows * pl.pw) * pl.tile_n;
        for (int s = 0; s < pl.num_stages; ++s) {
            uint8_t *e_tail = smem_raw + (smem_base - ptx::smem_u32(smem_raw)) + s * stage_bytes + pl.x_bytes +
                              pl.r_rows * pl.pw * pl.tile_n;
            for (int i = threadIdx.x * 16; i < tail_bytes; i += blockDim.x * 16)
                *reinterpret_cast<int4 *>(e_tail + i) = make_int4(0, 0, 0, 0);
        }
        ptx::fence_proxy_async();
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxStages; ++s) {
            ptx::mbar_init(full_bar(s), 1);
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
    const RoleCtx ctx{&abort_s, pl.dev};

    if (warp == 0) {
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0, inflight = 0, inflight_parity = 0;
            bool ok = true;
            for (int blk = blk_begin; blk < blk_end; ++blk) {
                if (!(ok = wait_bar<32>(empty_bar(stage), phase ^ 1u, ctx))) break;
                const int img = blk / pl.blocks_per_img, y0 = (blk % pl.blocks_per_img) * pl.r_rows;
                const uint32_t x_dst = smem_base + stage * stage_bytes, e_dst = x_dst + pl.x_bytes;
                ptx::mbar_expect_tx(full_bar(stage), (uint32_t)(pl.x_box_bytes + pl.e_box_bytes));
                // activation: columns -pad .. , rows y0 - pad .. ; error: columns 0 .. pw - 1 (zeros beyond wo), rows y0 ..
                ptx::tma_load_4d(x_dst, &map_x, full_bar(stage), c * pl.kc, -pl.pad, y0 - pl.pad, img);
                ptx::tma_load_4d(e_dst, &map_e, full_bar(stage), nt * pl.tile_n, 0, y0, img);
                inflight |= 1u << stage;
                inflight_parity = (inflight_parity & ~(1u << stage)) | (phase << stage);
                if (++stage == pl.num_stages) { stage = 0; phase ^= 1u; }
            }
            if (!ok)
                for (int s = 0; s < pl.num_stages; ++s)
                    if (inflight & (1u << s))
                        for (uint32_t i = 0; i < kSpinLimit; ++i)
                            if (ptx::mbar_try_wait(full_bar(s), (inflight_parity >> s) & 1u)) break;
        }
    } else if (warp == 1) {
        // the whole warp runs the issue loop; one elected lane issues the MMAs and commits (see elect_one)
        const uint32_t leader = elect_one();
        const uint32_t tmem_base = __shfl_sync(0xffffffffu, tmem_base_s, 0);
        const uint32_t idesc = make_idesc_i8(kTileM, pl.tile_n, true, true);
        // MN-major descriptors: activation atoms (taps) are one pixel (kc bytes) apart; 8-pixel groups 8 rows apart
        const uint32_t a_hi = smem_desc_hi(8u * pl.kc, layout_type_for(pl.kc));
        const uint32_t b_hi = smem_desc_hi(8u * pl.tile_n, layout_type_for(pl.tile_n));
        const uint32_t a_lead = ((uint32_t)pl.kc >> 4) << 16;
        const uint32_t a_step16 = (32u * pl.kc) >> 4, b_step16 = (32u * pl.tile_n) >> 4;  // 32 pixels further
        const uint32_t kc16 = (uint32_t)pl.kc >> 4, row16 = (uint32_t)(pl.pw * pl.kc) >> 4;
        // start offset of each accumulator's first tap inside the activation patch (16-byte units)
        uint32_t acc_off[kMaxAcc];
#pragma unroll
        for (int j = 0; j < kMaxAcc; ++j) {
            const int a = row0 + j / pl.accs_per_row, b0 = (j % pl.accs_per_row) * pl.apa;
            acc_off[j] = (uint32_t)a * row16 + (uint32_t)b0 * kc16;
        }
        const int k_steps = pl.kp / 32;
        int stage = 0;
        uint32_t phase = 0, accumulate = 0;
        bool ok = true;
        for (int it = 0; it < my_blocks; ++it) {
            if (!(ok = __all_sync(0xffffffffu, wait_bar(full_bar(stage), phase, ctx)))) break;
            ptx::tc_fence_after();
            uint32_t a_lo = ((smem_base + stage * stage_bytes) >> 4) | a_lead;
            uint32_t b_lo = (smem_base + stage * stage_bytes + pl.x_bytes) >> 4;
            for (int k = 0; k < k_steps; ++k) {
#pragma unroll
                for (int j = 0; j < kMaxAcc; ++j)
                    if (j < num_acc)
                        ptx::mma_i8(tmem_base + j * pl.tile_n, smem_desc_join(a_lo + acc_off[j], a_hi),
                                    smem_desc_join(b_lo, b_hi), idesc, accumulate, leader);
                accumulate = 1;
                a_lo += a_step16;
                b_lo += b_step16;
            }
            ptx::mma_commit(empty_bar(stage), leader);
            if (++stage == pl.num_stages) { stage = 0; phase ^= 1u; }
        }
        ptx::mma_commit(done_bar, leader);
        if (!ok)
            for (uint32_t i = 0; i < kSpinLimit; ++i)
                if (ptx::mbar_try_wait(done_bar, 0)) break;
    } else {
        const int quad = warp & 3;
        const int r = quad * 32 + lane;  // accumulator row: (tap within the accumulator, channel of the chunk)
        const int atom = r / pl.kc, ch = r % pl.kc;
        const bool ok = __all_sync(0xffffffffu, wait_bar<64>(done_bar, 0, ctx));
        int32_t *slice = pl.partials + (size_t)ks * pl.c_out * pl.rows_total;
        if (ok) {
            ptx::tc_fence_after();
            for (int j = 0; j < num_acc; ++j) {
                const int a = row0 + j / pl.accs_per_row, b = (j % pl.accs_per_row) * pl.apa + atom;
                const bool valid = b < pl.kdim;
                const size_t row = (size_t)(a * pl.kdim + b) * pl.c_in + c * pl.kc + ch;
                const uint32_t t_row = tmem_base + j * pl.tile_n + ((uint32_t)(quad * 32) << 16);
                for (int c0 = 0; c0 < pl.tile_n; c0 += 16) {
                    uint32_t v[32];
                    if (my_blocks > 0) {
                        ptx::tmem_ld_32x16(t_row + c0, v);
                        ptx::tmem_ld_wait();
                    } else {
#pragma unroll
                        for (int i = 0; i < 16; ++i) v[i] = 0;  // a CTA without pixel blocks still owns (zero) partials
                    }
                    if (valid) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            const int oc = nt * pl.tile_n + c0 + i;
                            slice[(size_t)oc * pl.rows_total + row] = (int32_t)v[i];
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

size_t wgrad_patch_smem_bytes(const WgradPatchPlan &pl)
{
    return (size_t)pl.num_stages * (pl.x_bytes + pl.e_bytes) + 1024;
}

cudaError_t launch_wgrad_patch(const WgradPatchPlan &pl, const CUtensorMap &map_x, const CUtensorMap &map_e,
                               cudaStream_t stream)
{
    cudaError_t e = cudaFuncSetAttribute(wgrad_patch_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 208 * 1024);
    if (e != cudaSuccess) return e;
    wgrad_patch_kernel<<<pl.num_groups * pl.num_splits, kWgradPatchThreads, wgrad_patch_smem_bytes(pl), stream>>>(pl, map_x,
                                                                                                                 map_e);
    return cudaGetLastError();
}

}  // namespace eoq
