// Patch variant of the implicit-GEMM convolution for stride-1 filters (forward pass and error back-propagation,
// arXiv 2105.13890, Sec. 3.2.1).
//
// The TMA engine of an SM delivers one row (<= 128 bytes) every ~4.7 cycles whatever the row width, so fetching
// every filter tap as its own 128-pixel tile makes a 3x3 layer load-bound at a fraction of the tensor rate.
// Here an M tile is `r_rows` whole output rows of one image, laid out in the raster of a source patch that is
// (k - 1) pixels wider than the output row.  The patch (with its zero halo, filled by the TMA out-of-bounds rule)
// is loaded ONCE per channel chunk; filter tap (a, b) is the same shared-memory tile read through a descriptor
// whose start address is (a * pw + b) rows further (the swizzle is a function of the address, so a row shift
// keeps operand and descriptor consistent).  Output rows that fall in the (k - 1) extra columns are computed and
// dropped.  Weights either stay resident in shared memory for the whole kernel (when the layer's weights fit) or
// stream through their own ring.
//
// Roles: warp 0 patch loads, warp 1 TMEM owner + tcgen05.mma issuer, warp 2 weight loads, warps 4-19 epilogue
// (four per TMEM lane quadrant: two pairs that take alternate tiles, the warps of a pair split the columns).
// All waits are bounded.
#include "eoq_device.cuh"
#include "eoq_epilogue.cuh"
#include "eoq_internal.h"

namespace eoq {

namespace {

constexpr int kMaxA = 4, kMaxB = 8;

__global__ void __launch_bounds__(kPatchThreads, 1)
igemm_patch_kernel(const __grid_constant__ IgemmParams p, const __grid_constant__ PatchPlan pl,
                   const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[2 * kMaxA + 2 * kMaxB + 5];
    __shared__ uint32_t tmem_base_s;
    __shared__ volatile uint32_t abort_s;

    const int warp = warp_index_uniform(), lane = threadIdx.x & 31;
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t b_sub = (uint32_t)p.tile_n * p.kc;
    const uint32_t b_region = smem_base + (uint32_t)pl.num_a * pl.a_bytes;
    const uint32_t table_off = (uint32_t)pl.num_a * pl.a_bytes + (pl.b_resident ? (uint32_t)pl.chunks * p.ntaps : (uint32_t)pl.num_b) * b_sub;
    const uint32_t bar0 = ptx::smem_u32(bars);
    auto a_full = [&](int s) { return bar0 + 8u * s; };
    auto a_empty = [&](int s) { return bar0 + 8u * (kMaxA + s); };
    auto b_full = [&](int s) { return bar0 + 8u * (2 * kMaxA + s); };
    auto b_empty = [&](int s) { return bar0 + 8u * (2 * kMaxA + kMaxB + s); };
    auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * kMaxA + 2 * kMaxB + a); };
    auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * kMaxA + 2 * kMaxB + 2 + a); };
    const uint32_t drain_bar = bar0 + 8u * (2 * kMaxA + 2 * kMaxB + 4);

    uint32_t acc_stride = 32;
    while (acc_stride < (uint32_t)p.tile_n) acc_stride <<= 1;
    // Tiles up to 128 columns keep two partial accumulators that successive MMAs alternate between (summed
    // exactly in the epilogue), which removes the wait of an MMA on its predecessor's write-back.
    const uint32_t nacc = p.tile_n <= 128 ? 2u : 1u;
    const uint32_t buf_stride = nacc * acc_stride;
    const uint32_t tmem_cols = 2 * buf_stride;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxA; ++s) {
            ptx::mbar_init(a_full(s), 1);
            ptx::mbar_init(a_empty(s), 1);
        }
        for (int s = 0; s < kMaxB; ++s) {
            ptx::mbar_init(b_full(s), 1);
            ptx::mbar_init(b_empty(s), 1);
        }
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(tfull_bar(a), 1);
            ptx::mbar_init(tempty_bar(a), kEpilogueWarps / 2);
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
    const int taps = p.ntaps;

    if (warp == 0) {
        if (lane == 0) {
            // ------------------------------------------------------------------ patch loads
            int ia = 0;
            uint32_t pha = 0, inflight = 0, inflight_parity = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                const int mt = tile / p.num_n_tiles;
                const int img = mt / pl.tiles_per_img, y0 = (mt % pl.tiles_per_img) * pl.r_rows;
                for (int c = 0; c < pl.chunks; ++c) {
                    if (!(ok = wait_bar<64>(a_empty(ia), pha ^ 1u, ctx))) break;
                    ptx::mbar_expect_tx(a_full(ia), (uint32_t)pl.a_box_bytes);
                    // source columns -pad .. -pad + pw - 1, rows y0 - pad .. : out-of-image pixels arrive as zeros
                    ptx::tma_load_4d(smem_base + ia * pl.a_bytes, &map_a, a_full(ia), c * p.kc, -pl.pad, y0 - pl.pad, img);
                    inflight |= 1u << ia;
                    inflight_parity = (inflight_parity & ~(1u << ia)) | (pha << ia);
                    if (++ia == pl.num_a) { ia = 0; pha ^= 1u; }
                }
            }
            if (!ok)
                for (int s = 0; s < pl.num_a; ++s)
                    if (inflight & (1u << s))
                        for (uint32_t i = 0; i < kSpinLimit; ++i)
                            if (ptx::mbar_try_wait(a_full(s), (inflight_parity >> s) & 1u)) break;
        }
    } else if (warp == 2) {
        if (lane == 0) {
            // ------------------------------------------------------------------ weight loads
            // One sub-tile = the weights of one tap for kc reduction channels and tile_n columns.  K-major: one box
            // [tile_n rows][kc bytes].  MN-major: tile_n / b_row boxes [kc rows][b_row bytes], one per atom.
            auto load_b = [&](uint32_t dst, uint32_t bar, int chunk, int tap, int n0) {
                if (!p.b_mn) {
                    ptx::tma_load_3d(dst, &map_b, bar, chunk * p.kc, tap, n0);
                } else {
                    const uint32_t atom = (uint32_t)p.kc * p.b_row;
                    for (int a = 0, na = p.tile_n / p.b_row; a < na; ++a)
                        ptx::tma_load_3d(dst + a * atom, &map_b, bar, n0 + a * p.b_row, tap, chunk * p.kc);
                }
            };
            if (pl.b_resident) {
                ptx::mbar_expect_tx(b_full(0), (uint32_t)pl.chunks * taps * b_sub);
                for (int c = 0; c < pl.chunks; ++c)
                    for (int t = 0; t < taps; ++t)
                        load_b(b_region + (c * taps + t) * b_sub, b_full(0), c, (int)p.tap_b[t], 0);
                // completion is observed by the MMA thread, which every path out of this kernel waits for
            } else {
                int ib = 0;
                uint32_t phb = 0, inflight = 0, inflight_parity = 0;
                bool ok = true;
                for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                    const int nt = tile % p.num_n_tiles;
                    for (int c = 0; c < pl.chunks && ok; ++c)
                        for (int t = 0; t < taps; ++t) {
                            if (!(ok = wait_bar<64>(b_empty(ib), phb ^ 1u, ctx))) break;
                            ptx::mbar_expect_tx(b_full(ib), b_sub);
                            load_b(b_region + ib * b_sub, b_full(ib), c, (int)p.tap_b[t], nt * p.tile_n);
                            inflight |= 1u << ib;
                            inflight_parity = (inflight_parity & ~(1u << ib)) | (phb << ib);
                            if (++ib == pl.num_b) { ib = 0; phb ^= 1u; }
                        }
                }
                if (!ok)
                    for (int s = 0; s < pl.num_b; ++s)
                        if (inflight & (1u << s))
                            for (uint32_t i = 0; i < kSpinLimit; ++i)
                                if (ptx::mbar_try_wait(b_full(s), (inflight_parity >> s) & 1u)) break;
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------------- MMA issuer (whole warp, see elect_one)
        const uint32_t leader = elect_one();
        const uint32_t tmem_base = __shfl_sync(0xffffffffu, tmem_base_s, 0);
        const uint32_t idesc = make_idesc_i8(kTileM, p.tile_n, false, p.b_mn != 0);
        const uint32_t hi = smem_desc_hi(8u * p.kc, layout_type_for(p.kc));
        // B: K-major like A, or MN-major atoms (swizzled rows: atoms kc * b_row apart along the columns = leading
        // offset, 8-row groups 8 * b_row apart = stride offset; 16-byte rows carry no swizzle and the two offsets
        // swap roles); a 32-deep K step is 32 bytes along a K-major row, 32 rows of an MN-major atom
        uint32_t b_hi = hi, b_k16 = 2u, b_lead = 0u;
        if (p.b_mn) {
            const uint32_t atom = (uint32_t)p.kc * p.b_row;
            if (p.b_row == 16) {
                b_hi = smem_desc_hi(atom, 0);
                b_lead = (128u >> 4) << 16;
            } else {
                b_hi = smem_desc_hi(8u * p.b_row, layout_type_for(p.b_row));
                b_lead = ((atom >> 4) & 0x3FFFu) << 16;
            }
            b_k16 = (32u * p.b_row) >> 4;
        }
        const uint32_t b_sub16 = b_sub >> 4, b_ring_lo = (b_region >> 4) | b_lead;
        const uint32_t kc16 = (uint32_t)p.kc >> 4, row16 = (uint32_t)(pl.pw * p.kc) >> 4;  // one pixel / one patch row
        const int k_steps = p.kc / 32, kdim = pl.kdim, chunks = pl.chunks, num_a = pl.num_a, num_b = pl.num_b;
        const bool resident = pl.b_resident != 0;
        int ia = 0, ib = 0, acc = 0;
        uint32_t pha = 0, phb = 0, acc_phase = 0;
        bool ok = true;
        if (resident) ok = __all_sync(0xffffffffu, wait_bar(b_full(0), 0, ctx));
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
            if (!(ok = __all_sync(0xffffffffu, wait_bar(tempty_bar(acc), acc_phase ^ 1u, ctx)))) break;
            ptx::tc_fence_after();
            uint32_t d0 = tmem_base + acc * buf_stride, d1 = nacc == 2 ? d0 + acc_stride : d0;
            const bool two_acc = nacc == 2;
            uint32_t b_res_lo = b_ring_lo;  // resident weights: walks (chunk, tap) sub-tiles in order
            uint32_t parity = 0;            // index of the next MMA of this tile, modulo 2 (generic path)
            bool fresh0 = true, fresh1 = two_acc;
            for (int c = 0; c < chunks && ok; ++c) {
                if (!(ok = __all_sync(0xffffffffu, wait_bar(a_full(ia), pha, ctx)))) break;
                ptx::tc_fence_after();
                uint32_t a_row = (smem_base + ia * pl.a_bytes) >> 4;
                if (resident && kdim == 3) {
                    // common case, fully unrolled: 9 taps x k_steps MMAs
                    if (k_steps == 4) mma_patch_chunk<3, 4>(d0, d1, a_row, b_res_lo, row16, kc16, b_sub16, hi, idesc, c == 0, two_acc, leader, b_hi, b_k16);
                    else if (k_steps == 2) mma_patch_chunk<3, 2>(d0, d1, a_row, b_res_lo, row16, kc16, b_sub16, hi, idesc, c == 0, two_acc, leader, b_hi, b_k16);
                    else {
                        mma_patch_chunk<3, 1>(d0, d1, a_row, b_res_lo, row16, kc16, b_sub16, hi, idesc, c == 0, two_acc, leader, b_hi, b_k16);
                        const uint32_t t = d0; d0 = d1; d1 = t;  // 9 MMAs: the next chunk starts on the other accumulator
                    }
                    b_res_lo += 9 * b_sub16;
                } else {
                    // tap (a, b) reads the patch tile (a * pw + b) rows further
                    for (int a = 0; a < kdim && ok; ++a, a_row += row16) {
                        uint32_t a_tap = a_row;
                        for (int b = 0; b < kdim; ++b, a_tap += kc16) {
                            uint32_t b_lo;
                            if (resident) {
                                b_lo = b_res_lo;
                                b_res_lo += b_sub16;
                            } else {
                                if (!(ok = __all_sync(0xffffffffu, wait_bar(b_full(ib), phb, ctx)))) break;
                                ptx::tc_fence_after();
                                b_lo = b_ring_lo + ib * b_sub16;
                            }
                            if (k_steps == 4) mma_k_steps<4>(d0, d1, a_tap, b_lo, hi, idesc, parity, fresh0, fresh1, leader, b_hi, b_k16);
                            else if (k_steps == 2) mma_k_steps<2>(d0, d1, a_tap, b_lo, hi, idesc, parity, fresh0, fresh1, leader, b_hi, b_k16);
                            else mma_k_steps<1>(d0, d1, a_tap, b_lo, hi, idesc, parity, fresh0, fresh1, leader, b_hi, b_k16);
                            if (k_steps == 1) {
                                // one MMA per tap: it went to accumulator `parity`; for a single accumulator d0 == d1
                                if (parity == 0) fresh0 = false; else fresh1 = false;
                                parity ^= 1u;
                            } else {
                                fresh0 = false;
                                fresh1 = false;
                            }
                            if (!resident) {
                                ptx::mma_commit(b_empty(ib), leader);
                                if (++ib == num_b) { ib = 0; phb ^= 1u; }
                            }
                        }
                    }
                }
                ptx::mma_commit(a_empty(ia), leader);
                if (++ia == num_a) { ia = 0; pha ^= 1u; }
            }
            if (ok) ptx::mma_commit(tfull_bar(acc), leader);
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
        if (!ok) {
            ptx::mma_commit(drain_bar, leader);
            for (uint32_t i = 0; i < kSpinLimit; ++i)
                if (ptx::mbar_try_wait(drain_bar, 0)) break;
            if (pl.b_resident)
                for (uint32_t i = 0; i < kSpinLimit; ++i)
                    if (ptx::mbar_try_wait(b_full(0), 0)) break;
        }
    } else if (warp >= 4) {
        // ---------------------------------------------------------------------- epilogue
        // The four warps of a TMEM lane quadrant form two pairs; pair `grp` serves every second tile of this CTA
        // (the tiles whose sums sit in accumulator buffer `grp`), and the two warps of a pair split the columns.
        // Two tiles are therefore in the epilogue at the same time: while one pair waits for tensor-memory loads
        // or stores, the other has arithmetic to issue.  Everything that does not depend on the sums (pixel
        // index, border class, b1 table row, shortcut codes) is formed before the wait for the tile's MMAs.
        const int quad = warp & 3;
        const int ew = (warp - 4) >> 2;
        const int grp = ew & 1, part = ew >> 1;
        const int row = quad * 32 + lane;
        const int groups = p.tile_n / 16;
        constexpr int kParts = kEpilogueWarps / 8;
        const int g_begin = (groups * part) / kParts, g_end = (groups * (part + 1)) / kParts;
        const int yl = row / pl.pw, xx = row % pl.pw;  // position of this thread's row in the patch raster
        const bool fwd = p.epilogue == kEpiForward;
        const FwdScalars fs = fwd ? load_fwd_scalars(p) : FwdScalars{0, 0, 0};
        // the b1 table of the whole layer goes to shared memory (behind the operand buffers), once, times b1
        const int32_t *ts = fwd ? stage_b1_table(p, fs.b1, smem_raw + (smem_base - ptx::smem_u32(smem_raw)) + table_off,
                                                 (int)threadIdx.x - 128, 32 * kEpilogueWarps)
                                : nullptr;
        uint32_t acc_phase = 0, mx = 0, mx_masked = 0;
        const bool wide_out = (reinterpret_cast<uintptr_t>(p.acc_out) & 31) == 0;   // 256-bit stores of the exact sums
        bool ok = true;
        // (column tile, image, row tile in the image) of the current tile, carried from tile to tile: the step
        // between two tiles of this pair is constant, so its quotients are formed once instead of four integer
        // divisions per tile and warp
        const int tile0 = blockIdx.x + grp * gridDim.x, step = 2 * gridDim.x;
        int nt = tile0 % p.num_n_tiles, mt0 = tile0 / p.num_n_tiles;
        int img = mt0 / pl.tiles_per_img, ti = mt0 % pl.tiles_per_img;
        const int step_nt = step % p.num_n_tiles, step_mt = step / p.num_n_tiles;
        const int step_img = step_mt / pl.tiles_per_img, step_ti = step_mt % pl.tiles_per_img;
        for (int tile = tile0; tile < num_tiles && ok; tile += step) {
            const int y = ti * pl.r_rows + yl;
            const bool valid = yl < pl.r_rows && xx < p.wq && y < p.hq;
            size_t pix = 0;
            int cls = 0;
            if (valid) {
                pix = ((size_t)img * p.hq + y) * p.wq + xx;
                if (p.b1_table)
                    cls = border_class(y, p.hq, p.b1_nlo_h, p.b1_nhi_h, p.b1_nrc) * p.b1_ncc +
                          border_class(xx, p.wq, p.b1_nlo_w, p.b1_nhi_w, p.b1_ncc);
            }
            int col = nt * p.tile_n + g_begin * 16;
            size_t off = pix * p.N + col;
            const int4 zero4 = make_int4(0, 0, 0, 0);
            // the shortcut codes do not depend on the sums: the first group's are requested before the wait for the MMAs
            int4 sc = (fwd && valid && col < p.N && p.shortcut) ? __ldg(reinterpret_cast<const int4 *>(p.shortcut + off)) : zero4;
            const int32_t *tb = ts ? ts + cls * p.N + col : nullptr;
            const int32_t *tg = (!ts && p.b1_table) ? p.b1_table + (size_t)cls * p.N + col : nullptr;
            if (!(ok = __all_sync(0xffffffffu, wait_bar<64>(tfull_bar(grp), acc_phase, ctx)))) break;
            ptx::tc_fence_after();
            const uint32_t t_row = tmem_base + grp * buf_stride + ((uint32_t)(quad * 32) << 16);
            for (int g = g_begin; g < g_end; ++g, col += 16, off += 16) {
                uint32_t r[32];
                ptx::tmem_ld_32x16(t_row + g * 16, r);
                uint32_t r2[32];
                if (nacc == 2) ptx::tmem_ld_32x16(t_row + acc_stride + g * 16, r2);
                // the next group's shortcut codes travel while this group is computed
                int4 sc_next = zero4;
                if (g + 1 < g_end && fwd && valid && col + 16 < p.N && p.shortcut)
                    sc_next = __ldg(reinterpret_cast<const int4 *>(p.shortcut + off + 16));
                ptx::tmem_ld_wait();
                if (nacc == 2 && !fwd) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) r[i] += r2[i];  // the two partial accumulators of the tile
                }
                if (valid && col < p.N) {
                    if (fwd) {
                        if (nacc == 2) {
                            if (p.relu) forward_16<true, true, true>(p, fs, r, r2, off, tb, tg, sc, 7);
                            else forward_16<true, false, true>(p, fs, r, r2, off, tb, tg, sc, 7);
                        } else {
                            if (p.relu) forward_16<true, true, false>(p, fs, r, r2, off, tb, tg, sc, 7);
                            else forward_16<true, false, false>(p, fs, r, r2, off, tb, tg, sc, 7);
                        }
                    }
                    else mx = max(mx, wide_out ? dgrad_16<true>(p, r, off, mx_masked) : dgrad_16<false>(p, r, off, mx_masked));
                }
                sc = sc_next;
                if (tb) tb += 16;
                if (tg) tg += 16;
            }
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(tempty_bar(grp));
            acc_phase ^= 1u;
            nt += step_nt;
            ti += step_ti;
            if (nt >= p.num_n_tiles) { nt -= p.num_n_tiles; ++ti; }
            img += step_img;
            if (ti >= pl.tiles_per_img) { ti -= pl.tiles_per_img; ++img; }
            if (ti >= pl.tiles_per_img) { ti -= pl.tiles_per_img; ++img; }
        }
        if (p.epilogue == kEpiDgrad) {
            mx = warp_max_u32(mx);
            if (lane == 0 && mx) atomicMax(&p.dev->absmax_u32, mx);
            if (p.next_mask) {
                mx_masked = warp_max_u32(mx_masked);
                if (lane == 0 && mx_masked) atomicMax(&p.dev->absmax_u64, (unsigned long long)mx_masked);
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

size_t igemm_patch_smem_bytes(const IgemmParams &p, const PatchPlan &pl)
{
    const size_t b_sub = (size_t)p.tile_n * p.kc;
    const size_t b = pl.b_resident ? (size_t)pl.chunks * p.ntaps * b_sub : (size_t)pl.num_b * b_sub;
    return (size_t)pl.num_a * pl.a_bytes + b + 1024 + kTableSmemBytes;
}

cudaError_t launch_igemm_patch(const IgemmParams &p, const PatchPlan &pl, const CUtensorMap &map_a,
                               const CUtensorMap &map_b, int grid, cudaStream_t stream)
{
    cudaError_t e = cudaFuncSetAttribute(igemm_patch_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 226 * 1024);
    if (e != cudaSuccess) return e;
    igemm_patch_kernel<<<grid, kPatchThreads, igemm_patch_smem_bytes(p, pl), stream>>>(p, pl, map_a, map_b);
    return cudaGetLastError();
}

}  // namespace eoq
