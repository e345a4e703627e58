// eoq_conv_dgrad_static: error back-propagation for callers that cannot allocate device memory.
// All scratch (the reduction cells, the transposed weights, the int32 sums) lives in one file-scope device
// array that every GPU loading the library carries until the process exits.
#include <cuda_runtime.h>
#include <stdint.h>

#include <functional>
#include <mutex>

#include "eoq_internal.h"

using namespace eoq;

namespace {

constexpr size_t kStaticHeaderBytes = 4096;  // reduction cells and status word (a DeviceState)
constexpr size_t kStaticScratchBytes = (size_t)EOQ_STATIC_SCRATCH_BYTES;
static_assert(sizeof(DeviceState) <= kStaticHeaderBytes, "header too small");

// In host code this name is only a handle for the runtime: its device address comes from
// cudaGetSymbolAddress, once per device.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticHeaderBytes + kStaticScratchBytes];

constexpr int kMaxDevices = 64;
struct PerDevice {
    std::once_flag once;     // the set-up runs once per device even when several host threads make the first call together
    int setup_status;        // EOQ_OK, or why the set-up failed
    unsigned char *scratch;  // device address of g_static_scratch on this device
    int sm_count;
};
PerDevice g_per_device[kMaxDevices];
int g_last_cuda_error = 0;   // last cudaError_t of the allocation-free path (eoq_last_cuda_error(NULL) returns it)

int fail(cudaError_t e)
{
    g_last_cuda_error = (int)e;
    return EOQ_ERR_CUDA;
}

// First call on a device: resolves the array's device address and reads two attributes.  Nothing is allocated here,
// but the CUDA module that holds the array is loaded at the latest now, and the driver reserves the array's memory
// with it: on a device that is already full this is where cudaErrorMemoryAllocation shows up.
void setup_device(PerDevice &pd, int device)
{
    void *ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (e != cudaSuccess || !ptr) { pd.setup_status = fail(e != cudaSuccess ? e : cudaErrorInvalidSymbol); return; }
    int sms = 0, major = 0;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device)) != cudaSuccess ||
        (e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device)) != cudaSuccess) {
        pd.setup_status = fail(e);
        return;
    }
    if (major != 10) { pd.setup_status = EOQ_ERR_UNSUPPORTED; return; }
    pd.scratch = static_cast<unsigned char *>(ptr);
    pd.sm_count = sms;
    pd.setup_status = EOQ_OK;
}

}  // namespace

extern "C" int eoq_conv_dgrad_static(const eoq_conv_desc_t *desc, const int8_t *e3, const int32_t *e3_exp,
                                     const int8_t *w, int8_t *e4, int32_t *e4_exp, int64_t *sum_e4,
                                     uint32_t *status_out, void *stream)
{
    int device = -1;
    cudaError_t ce = cudaGetDevice(&device);
    if (ce != cudaSuccess || device < 0 || device >= kMaxDevices) return fail(ce != cudaSuccess ? ce : cudaErrorInvalidDevice);
    PerDevice &pd = g_per_device[device];
    std::call_once(pd.once, setup_device, std::ref(pd), device);
    if (pd.setup_status != EOQ_OK) return pd.setup_status;
    size_t need = 0;
    int st = eoq_workspace_size(desc, EOQ_PASS_DGRAD, &need);
    if (st != EOQ_OK) return st;
    if (need > kStaticScratchBytes) return EOQ_ERR_WORKSPACE;  // geometry needs more scratch than the array holds

    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    // the array keeps what the previous call left: the status word and the cells must start at zero
    if ((ce = cudaMemsetAsync(pd.scratch, 0, sizeof(DeviceState), s)) != cudaSuccess) return fail(ce);

    Handle h;  // host-side bookkeeping only; its device state is the head of the static array
    h.device = device;
    h.sm_count = pd.sm_count;
    h.last_cuda_error = 0;
    h.dev = reinterpret_cast<DeviceState *>(pd.scratch);
    h.launches = 0;
    h.profiling = false;
    h.force_timeout = false;
    h.gemm_only = false;
    h.hook = ReduceHook{nullptr, nullptr};
    h.num_records = 0;
    h.records = nullptr;
    h.gemm_ctas = pd.sm_count;
    h.fork_ev = h.join_ev = nullptr;
    for (int k = 0; k < kClassBranches; ++k) {
        h.class_branch[k] = nullptr;
        h.class_join[k] = nullptr;
    }
    st = eoq_conv_dgrad(reinterpret_cast<eoq_handle_t>(&h), desc, e3, e3_exp, w, e4, e4_exp, sum_e4, nullptr,
                        pd.scratch + kStaticHeaderBytes, kStaticScratchBytes, stream);
    if (st != EOQ_OK) {
        if (st == EOQ_ERR_CUDA) g_last_cuda_error = h.last_cuda_error;
        return st;
    }
    if (status_out && (ce = cudaMemcpyAsync(status_out, pd.scratch + offsetof(DeviceState, status), sizeof(uint32_t),
                                            cudaMemcpyDeviceToDevice, s)) != cudaSuccess)
        return fail(ce);
    return EOQ_OK;
}

namespace eoq {
int static_path_last_cuda_error() { return g_last_cuda_error; }
}  // namespace eoq
