// placeholder until the tcgen05 kernel lands
#include "common.cuh"
namespace rmsmp {
bool tensor_supported(const Problem&) { return false; }
rmsmp_status launch_tensor(const Problem&, cudaStream_t) { return RMSMP_ERR_VARIANT; }
}
