// Implicit-GEMM convolution kernel for sm_100a: forward pass and error back-propagation of the EOQ layer
// (arXiv 2105.13890, Sec. 3.2.1).  One persistent CTA per SM walks 128-row output tiles:
//   warps 0, 2, 3: TMA producers (im2col loads of the activation/error operand, tiled loads of the weights); a
//              thread gets a TMA instruction out only every few hundred cycles, but threads of different warps
//              issue side by side, so the pipeline stages rotate over three producers
//   warp 1       : owns tensor memory, issues tcgen05.mma kind::i8 (int8 x int8 -> int32 in TMEM)
//   warps 4-19   : epilogue; read the accumulators with tcgen05.ld and apply the layer's quantizers in registers
// Two accumulator buffers in TMEM let the epilogue of tile i overlap the main loop of tile i+1.
// Every wait is bounded: when one runs out the CTA raises EOQ_DEV_TIMEOUT, drains and returns.
#include "eoq_device.cuh"
#include "eoq_epilogue.cuh"
#include "eoq_internal.h"

namespace eoq {

namespace {

constexpr int kMaxStages = 8;
constexpr int kProducers = 3;

__global__ void __launch_bounds__(kGemmThreads, 1)
igemm_kernel(const __grid_constant__ IgemmParams p, const __grid_constant__ CUtensorMap map_a,
             const __grid_constant__ CUtensorMap map_b)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[2 * kMaxStages + 5];
    __shared__ uint32_t tmem_base_s;
    __shared__ volatile uint32_t abort_s;

    const int warp = warp_index_uniform(), lane = threadIdx.x & 31;
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
    // Tiles up to 128 columns keep two partial accumulators that successive MMAs alternate between (summed
    // exactly in the epilogue), which removes the wait of an MMA on its predecessor's write-back.
    const uint32_t nacc = (p.tile_n <= 128 && p.kc >= 32 && p.num_sub * (p.kc / 32) >= 2) ? 2u : 1u;
    const uint32_t buf_stride = nacc * acc_stride;
    const uint32_t tmem_cols = 2 * buf_stride;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.num_stages; ++s) {
            ptx::mbar_init(full_bar(s), 1);
            ptx::mbar_init(empty_bar(s), 1);
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
    const int k_iters = (p.num_sub + p.subs_per_stage - 1) / p.subs_per_stage;
    const int pix_per_img = p.hq * p.wq;

    if (warp == 0 || warp == 2 || warp == 3) {
        if (lane == 0) {
            // ------------------------------------------------------------------ TMA producers
            // producer q fills the pipeline slots q, q + 3, q + 6, ... of the CTA's sequence of (tile, k iteration)
            const int q = warp == 0 ? 0 : warp - 1;
            int stage = q % p.num_stages;
            uint32_t phase = (uint32_t)(q / p.num_stages) & 1u;
            int turn = q;  // slots until this producer's next one
            uint32_t inflight = 0, inflight_parity = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                const int mt = tile / p.num_n_tiles, nt = tile % p.num_n_tiles;
                const int m0 = mt * kTileM;
                const int img = m0 / pix_per_img, rem = m0 % pix_per_img;
                const int cw = (rem % p.wq) * p.src_stride_w + p.base_w;
                const int ch = (rem / p.wq) * p.src_stride + p.base_h;
                for (int kit = 0; kit < k_iters; ++kit) {
                    if (turn-- != 0) continue;
                    turn = kProducers - 1;
                    if (!(ok = wait_bar<32>(empty_bar(stage), phase ^ 1u, ctx))) break;
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
                        if (p.b_mn) {
                            // weights in place, [reduction rows][tap][columns]: tile_n / b_row atoms of [kc rows][b_row bytes]
                            const uint32_t atom = (uint32_t)p.kc * p.b_row;
                            for (int a = 0, na = p.tile_n / p.b_row; a < na; ++a)
                                ptx::tma_load_3d(b_dst + j * b_sub + a * atom, &map_b, full_bar(stage),
                                                 nt * p.tile_n + a * p.b_row, (int)p.tap_b[tap], chunk * p.kc);
                        } else {
                            // tap coordinate p.ntaps lies outside the weight tensor: the padding sub-tile is zero-filled
                            ptx::tma_load_3d(b_dst + j * b_sub, &map_b, full_bar(stage), chunk * p.kc,
                                             s < p.real_sub ? (int)p.tap_b[tap] : 0x7fff, nt * p.tile_n);
                        }
                    }
                    inflight |= 1u << stage;
                    inflight_parity = (inflight_parity & ~(1u << stage)) | (phase << stage);
                    stage += kProducers;
                    while (stage >= p.num_stages) { stage -= p.num_stages; phase ^= 1u; }
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
        // the whole warp runs the issue loop; one elected lane issues the MMAs and commits (see elect_one)
        const uint32_t leader = elect_one();
        const uint32_t tmem_base = __shfl_sync(0xffffffffu, tmem_base_s, 0);
        // ------------------------------------------------------------------ MMA issuer
        const uint32_t idesc = make_idesc_i8(kTileM, p.tile_n, false, p.b_mn != 0);
        // Descriptors are assembled from precomputed halves; the loop only adds offsets in 16-byte units.
        // kc >= 32: swizzled K-major sub-tiles, rows kc bytes wide, 8-row groups 8*kc apart; a 32-byte K step
        // moves the start address inside the swizzle span.  kc == 16: no swizzle, one MMA spans two sub-tiles
        // (two taps): the second half of K sits one sub-tile further (leading offset), 8-row groups 128 B apart.
        const bool wide = p.kc >= 32;
        const uint32_t hi = wide ? smem_desc_hi(8u * p.kc, layout_type_for(p.kc)) : smem_desc_hi(128, 0);
        const uint32_t a_sub16 = a_sub >> 4, b_sub16 = b_sub >> 4;
        const uint32_t a_lead = wide ? 0u : (a_sub16 << 16);
        uint32_t b_lead = wide ? 0u : (b_sub16 << 16);
        // B read MN-major (only with kc >= 32): atoms kc * b_row apart along the columns (leading offset), 8-row
        // groups 8 * b_row apart (stride offset); 16-byte rows carry no swizzle and the two offsets swap roles; a
        // 32-deep K step is 32 rows of an atom
        uint32_t b_hi = hi, b_k16 = 2u;
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
        const int sub_step = wide ? 1 : 2, k_steps = wide ? p.kc / 32 : 1;
        int stage = 0, acc = 0;
        uint32_t phase = 0, acc_phase = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
            if (!(ok = __all_sync(0xffffffffu, wait_bar(tempty_bar(acc), acc_phase ^ 1u, ctx)))) break;
            ptx::tc_fence_after();
            const uint32_t d_tmem = tmem_base + acc * buf_stride, d_other = nacc == 2 ? d_tmem + acc_stride : d_tmem;
            uint32_t accumulate = 0;
            uint32_t fresh0 = 1u, fresh1 = nacc == 2 ? 1u : 0u;
            for (int kit = 0; kit < k_iters; ++kit) {
                if (!(ok = __all_sync(0xffffffffu, wait_bar(full_bar(stage), phase, ctx)))) break;
                ptx::tc_fence_after();
                const int subs = min(p.subs_per_stage, p.num_sub - kit * p.subs_per_stage);
                uint32_t a_lo = ((smem_base + stage * stage_bytes) >> 4) | a_lead;
                uint32_t b_lo = (((smem_base + stage * stage_bytes) >> 4) + p.subs_per_stage * a_sub16) | b_lead;
                if (wide && k_steps >= 2) {
                    // 2 or 4 MMAs per sub-tile, alternating between the two partial accumulators
                    for (int j = 0; j < subs; ++j) {
                        if (k_steps == 4) mma_k_steps<4>(d_tmem, d_other, a_lo, b_lo, hi, idesc, 0, fresh0, fresh1, leader, b_hi, b_k16);
                        else mma_k_steps<2>(d_tmem, d_other, a_lo, b_lo, hi, idesc, 0, fresh0, fresh1, leader, b_hi, b_k16);
                        fresh0 = 0;
                        fresh1 = 0;
                        a_lo += a_sub16;
                        b_lo += b_sub16;
                    }
                } else {
                    for (int j = 0; j < subs; j += sub_step) {
                        // one MMA per step; with two accumulators successive steps alternate
                        const bool odd = nacc == 2 && (accumulate & 2u);
                        ptx::mma_i8(odd ? d_other : d_tmem, smem_desc_join(a_lo, hi), smem_desc_join(b_lo, b_hi), idesc,
                                    odd ? (fresh1 ? 0u : 1u) : (fresh0 ? 0u : 1u), leader);
                        if (odd) fresh1 = 0; else fresh0 = 0;
                        if (nacc == 2) accumulate ^= 2u;
                        a_lo += sub_step * a_sub16;
                        b_lo += sub_step * b_sub16;
                    }
                }
                ptx::mma_commit(empty_bar(stage), leader);
                if (++stage == p.num_stages) { stage = 0; phase ^= 1u; }
            }
            if (ok) ptx::mma_commit(tfull_bar(acc), leader);
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
        if (!ok) {
            ptx::mma_commit(drain_bar, leader);
            for (uint32_t i = 0; i < kSpinLimit; ++i)
                if (ptx::mbar_try_wait(drain_bar, 0)) break;
        }
    } else {
        // ---------------------------------------------------------------------- epilogue
        // A warp may read the TMEM lanes of quadrant (warp % 4).  The four warps of a quadrant form two pairs;
        // pair `grp` serves every second tile of this CTA (accumulator buffer `grp`), the two warps of a pair
        // split the tile's columns, so that two tiles are in the epilogue at the same time.  Everything that does
        // not depend on the sums is formed before the wait for the tile's MMAs.
        const int quad = warp & 3;
        const int ew = (warp - 4) >> 2;
        const int grp = ew & 1, part = ew >> 1;
        const int row = quad * 32 + lane;
        const int groups = p.tile_n / 16;                 // 16-column groups of the tile
        constexpr int kParts = kEpilogueWarps / 8;
        const int g_begin = (groups * part) / kParts, g_end = (groups * (part + 1)) / kParts;
        const bool fwd = p.epilogue == kEpiForward;
        const FwdScalars fs = fwd ? load_fwd_scalars(p) : FwdScalars{0, 0, 0};
        // the b1 table of the whole layer goes to shared memory (behind the pipeline stages), once, times b1
        const int32_t *ts = fwd ? stage_b1_table(p, fs.b1, smem_raw + (smem_base - ptx::smem_u32(smem_raw)) + p.num_stages * stage_bytes,
                                                 (int)threadIdx.x - 128, 32 * kEpilogueWarps)
                                : nullptr;
        int shift = 7;
        if (fwd && p.x_exp) {
            shift = -__ldg(p.x_exp);
            if (shift > 31 || shift < -16) {
                if (lane == 0) atomicOr(&p.dev->status, EOQ_DEV_RANGE);
                shift = max(-16, min(31, shift));
            }
        }
        uint32_t acc_phase = 0, mx = 0, mx_masked = 0;
        const bool wide_out = (reinterpret_cast<uintptr_t>(p.acc_out) & 31) == 0;   // 256-bit stores of the exact sums
        bool ok = true;
        for (int tile = blockIdx.x + grp * gridDim.x; tile < num_tiles && ok; tile += 2 * gridDim.x) {
            const int mt = tile / p.num_n_tiles, nt = tile % p.num_n_tiles;
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
            int col = nt * p.tile_n + g_begin * 16;
            size_t off = pix * p.N + col;
            const int4 zero4 = make_int4(0, 0, 0, 0);
            // the shortcut codes do not depend on the sums: the first group's are requested before the wait for the MMAs
            int4 sc = (fwd && valid && col < p.N && p.shortcut) ? __ldg(reinterpret_cast<const int4 *>(p.shortcut + off)) : zero4;
            const int32_t *tb = ts ? ts + cls * p.N + col : nullptr;
            const int32_t *tg = (!ts && p.b1_table) ? p.b1_table + (size_t)cls * p.N + col : nullptr;
            if (!(ok = __all_sync(0xffffffffu, wait_bar(tfull_bar(grp), acc_phase, ctx)))) break;  // warp-uniform
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
                        if (shift == 7) {
                            if (nacc == 2) {
                                if (p.relu) forward_16<true, true, true>(p, fs, r, r2, off, tb, tg, sc, 7);
                                else forward_16<true, false, true>(p, fs, r, r2, off, tb, tg, sc, 7);
                            } else {
                                if (p.relu) forward_16<true, true, false>(p, fs, r, r2, off, tb, tg, sc, 7);
                                else forward_16<true, false, false>(p, fs, r, r2, off, tb, tg, sc, 7);
                            }
                        } else {
                            // the generic shift (first layer behind the input quantizer) merges the partial sums itself
                            if (nacc == 2) {
#pragma unroll
                                for (int i = 0; i < 16; ++i) r[i] += r2[i];
                            }
                            if (p.relu) forward_16<false, true, false>(p, fs, r, r2, off, tb, tg, sc, shift);
                            else forward_16<false, false, false>(p, fs, r, r2, off, tb, tg, sc, shift);
                        }
                    } else {
                        mx = max(mx, wide_out ? dgrad_16<true>(p, r, off, mx_masked) : dgrad_16<false>(p, r, off, mx_masked));
                    }
                }
                sc = sc_next;
                if (tb) tb += 16;
                if (tg) tg += 16;
            }
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(tempty_bar(grp));
            acc_phase ^= 1u;
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

size_t igemm_smem_bytes(const IgemmParams &p)
{
    return (size_t)p.num_stages * p.subs_per_stage * ((size_t)kTileM + p.tile_n) * p.kc + 1024 + kTableSmemBytes;
}

cudaError_t launch_igemm(const IgemmParams &p, const CUtensorMap &map_a, const CUtensorMap &map_b, int grid,
                         cudaStream_t stream)
{
    const size_t smem = igemm_smem_bytes(p);
    cudaError_t e = cudaFuncSetAttribute(igemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 226 * 1024);
    if (e != cudaSuccess) return e;
    igemm_kernel<<<grid, kGemmThreads, smem, stream>>>(p, map_a, map_b);
    return cudaGetLastError();
}

}  // namespace eoq
