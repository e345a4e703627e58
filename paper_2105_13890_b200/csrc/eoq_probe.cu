// Issue-rate measurement of tcgen05.mma kind::i8 (the instruction every convolution pass of the library runs on):
// what the tensor pipe of this GPU delivers when nothing else is in the way.  Both operands are resident in shared
// memory (filled once by the CTA's own threads, no loads in the timed loop), accumulators live in tensor memory,
// one CTA per SM, one warp issues `iters` rounds of four 128 x N x 32 MMAs that alternate between two accumulators
// (as the convolution kernels do).  The only wait, for the last MMA, is bounded.
#include <cuda_runtime.h>
#include <stdint.h>

#include "eoq_device.cuh"
#include "eoq_internal.h"

namespace eoq {

namespace {

constexpr int kProbeThreads = 128;

__global__ void __launch_bounds__(kProbeThreads, 1)
probe_mma_i8_kernel(int n_cols, int iters, DeviceState *dev, unsigned long long *cycles_out)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t done_bar_s;
    __shared__ uint32_t tmem_base_s;
    const int warp = warp_index_uniform(), lane = threadIdx.x & 31;
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *base = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
    // A: 128 rows x 128 bytes, B: n_cols rows x 128 bytes (K-major, 128-byte swizzle atoms; the swizzle permutes
    // 16-byte chunks inside an 8-row group, which leaves a random fill random).  Values shaped like the layer's
    // operands: post-ReLU activation codes (half zeros) against small weight codes.
    const int a_bytes = kTileM * 128, b_bytes = n_cols * 128;
    for (int i = threadIdx.x; i < a_bytes + b_bytes; i += blockDim.x) {
        uint32_t h = (uint32_t)i * 2654435761u + blockIdx.x * 40503u;
        h ^= h >> 15;
        h *= 2246822519u;
        h ^= h >> 13;
        int v;
        if (i < a_bytes) v = (h & 1u) ? (int)((h >> 8) % 97u) : 0;
        else v = (int)((h >> 8) % 7u) - 3;
        base[i] = (uint8_t)(int8_t)v;
    }
    ptx::fence_proxy_async();
    uint32_t acc_stride = 32;
    while (acc_stride < (uint32_t)n_cols) acc_stride <<= 1;
    const uint32_t tmem_cols = 2 * acc_stride;
    if (threadIdx.x == 0) {
        ptx::mbar_init(ptx::smem_u32(&done_bar_s), 1);
        ptx::fence_barrier_init();
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(&tmem_base_s), tmem_cols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;
    if (warp == 1) {
        const uint32_t leader = elect_one();
        const uint32_t idesc = make_idesc_i8(kTileM, n_cols, false, false);
        const uint32_t hi = smem_desc_hi(8u * 128u, layout_type_for(128));
        const uint32_t a_lo = smem_base >> 4, b_lo = (smem_base + a_bytes) >> 4;
        const uint32_t d0 = tmem_base, d1 = tmem_base + acc_stride;
        const long long t0 = clock64();
        for (int it = 0; it < iters; ++it)
            mma_k_steps<4>(d0, d1, a_lo, b_lo, hi, idesc, 0, it == 0 ? 1u : 0u, it == 0 ? 1u : 0u, leader, hi, 2u);
        ptx::mma_commit(ptx::smem_u32(&done_bar_s), leader);
        bool ok = false;
        for (uint32_t i = 0; i < kSpinLimit; ++i)
            if (ptx::mbar_try_wait(ptx::smem_u32(&done_bar_s), 0)) { ok = true; break; }
        const long long t1 = clock64();
        if (lane == 0) {
            if (!ok) atomicOr(&dev->status, EOQ_DEV_TIMEOUT);
            if (cycles_out) atomicMax(cycles_out, (unsigned long long)(t1 - t0));
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

cudaError_t launch_probe_mma_i8(int n_cols, int iters, int grid, DeviceState *dev, unsigned long long *cycles_out,
                                cudaStream_t s)
{
    const size_t smem = (size_t)(kTileM + n_cols) * 128 + 1024;
    cudaError_t e = cudaFuncSetAttribute(probe_mma_i8_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    probe_mma_i8_kernel<<<grid, kProbeThreads, smem, s>>>(n_cols, iters, dev, cycles_out);
    return cudaGetLastError();
}

}  // namespace eoq
