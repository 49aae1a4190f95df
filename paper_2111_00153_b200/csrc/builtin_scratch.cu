// rmsmp_gemm_builtin_scratch: the workspace variant of the linear layer for callers that have
// no scratch buffer to give and no way to get one.
//
// Some users of this library run where device memory cannot be allocated at call time: inside
// a plugin of a serving runtime that hands out a fixed arena and forbids cudaMalloc, in a
// real-time loop where an allocation's implicit synchronisation is not acceptable, or after
// the process has been told to stay within the memory it already holds.  For them the scratch
// the workspace variant needs lives in this file, in device memory that belongs to the loaded
// library itself.
#include <cuda_runtime.h>
#include <atomic>
#include "common.cuh"

namespace {

// Scratch for the expanded (int8) weights of ONE layer.  4 MiB covers M * Kp of every layer of
// ResNet-18 (512 x 4608) and of BERT-base / BERT-large (4096 x 1024).  Every GPU that loads the
// library holds these bytes until the process exits.
constexpr size_t kBuiltinScratchBytes = 4u << 20;
static __device__ __align__(256) unsigned char g_builtin_scratch[kBuiltinScratchBytes];

// In host code `g_builtin_scratch` is only a handle for the runtime, not a device address; the
// address each device gave the array is looked up once per device and kept here.
// Host threads may make their first call on a device at the same time; the slot is an atomic pointer
// (every thread that looks the address up gets the same answer, so a lost race costs one more lookup).
std::atomic<void*> g_scratch_ptr[rmsmp::kMaxDevices];

rmsmp_status scratch_address(void** out)
{
    const int dev = rmsmp::device_ordinal();
    if (dev < 0) return RMSMP_ERR_CUDA;
    void* ptr = g_scratch_ptr[dev].load(std::memory_order_acquire);
    if (!ptr) {
        // With lazy module loading this lookup is also what makes the driver place the array on the device.
        if (cudaGetSymbolAddress(&ptr, g_builtin_scratch) != cudaSuccess || ptr == nullptr) {
            cudaGetLastError();
            return RMSMP_ERR_CUDA;
        }
        g_scratch_ptr[dev].store(ptr, std::memory_order_release);
    }
    *out = ptr;
    return RMSMP_OK;
}

}  // namespace

extern "C" rmsmp_status rmsmp_gemm_builtin_scratch(const rmsmp_layer* layer, const void* d_packed,
                                                   const int8_t* d_act, int64_t N, int64_t ld_act,
                                                   float act_step, float* d_out, int64_t ld_out,
                                                   rmsmp_out_layout out_layout, int32_t* d_acc,
                                                   void* stream)
{
    size_t need = 0;
    rmsmp_status st = rmsmp_workspace_bytes(layer, &need);     // also checks the descriptor
    if (st != RMSMP_OK) return st;
    if ((size_t)layer->M * (size_t)layer->Kp > kBuiltinScratchBytes) return RMSMP_ERR_BUFFER_TOO_SMALL;
    void* scratch = nullptr;
    st = scratch_address(&scratch);
    if (st != RMSMP_OK) return st;
    // Everything about the contraction is checked BEFORE the expansion is queued: a call that is going
    // to be refused must not touch the shared array, which an earlier call's kernels may still be reading.
    rmsmp::Problem p;
    st = rmsmp::gemm_prepare(layer, d_packed, scratch, true, d_act, N, ld_act, act_step, d_out, ld_out, out_layout,
                             d_acc, nullptr, p);
    if (st != RMSMP_OK) return st;
    if (!rmsmp::tensor_supported(p)) return RMSMP_ERR_VARIANT;
    // The expansion rewrites every byte the contraction will read (M rows of Kp bytes), so what an
    // earlier call left in the array never matters and nothing needs clearing.
    st = rmsmp_expand_weights(layer, d_packed, scratch, kBuiltinScratchBytes, stream);
    if (st != RMSMP_OK) return st;
    return rmsmp::dispatch_problem(p, RMSMP_VARIANT_TENSOR, static_cast<cudaStream_t>(stream));
}
