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
#include "common.cuh"

namespace {

// Scratch for the expanded (int8) weights of ONE layer.  4 MiB covers M * Kp of every layer of
// ResNet-18 (512 x 4608) and of BERT-base / BERT-large (4096 x 1024).  Every GPU that loads the
// library holds these bytes until the process exits.
constexpr size_t kBuiltinScratchBytes = 4u << 20;
static __device__ __align__(256) unsigned char g_builtin_scratch[kBuiltinScratchBytes];

// In host code `g_builtin_scratch` is only a handle for the runtime, not a device address; the
// address each device gave the array is looked up once per device and kept here.
void* g_scratch_ptr[64];
bool g_scratch_known[64];

rmsmp_status scratch_address(void** out)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        cudaGetLastError();
        return RMSMP_ERR_CUDA;
    }
    if (!g_scratch_known[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_builtin_scratch) != cudaSuccess || ptr == nullptr) {
            cudaGetLastError();
            return RMSMP_ERR_CUDA;
        }
        g_scratch_ptr[dev] = ptr;
        g_scratch_known[dev] = true;
    }
    *out = g_scratch_ptr[dev];
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
    // The expansion rewrites every byte the contraction will read (M rows of Kp bytes), so what an
    // earlier call left in the array never matters and nothing needs clearing.
    st = rmsmp_expand_weights(layer, d_packed, scratch, kBuiltinScratchBytes, stream);
    if (st != RMSMP_OK) return st;
    return rmsmp_gemm_workspace(layer, d_packed, scratch, d_act, N, ld_act, act_step, d_out, ld_out,
                                out_layout, d_acc, stream);
}
