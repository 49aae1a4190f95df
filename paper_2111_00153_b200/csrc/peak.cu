// Tensor-pipe ceiling of this GPU for the MMA shape the contraction kernel uses: every SM issues
// tcgen05.mma (M=128, N=256) back to back on operands that stay in shared memory -- no loads, no
// epilogue.  kind::i8 (K=32 per instruction) gives the INT8 roofline the layer kernels are measured
// against; kind::f16 with bf16 operands (K=16) calibrates it against the known bf16 figure.
#include <cuda.h>
#include "common.cuh"
#include "ptx.cuh"

namespace rmsmp {
namespace {

constexpr int kPeakThreads = 128;
constexpr int kPeakSmem = 16384 + 32768 + 1024 + 64;

__device__ __forceinline__ uint32_t pk_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__global__ void __launch_bounds__(kPeakThreads, 1) mma_peak_kernel(int is_bf16, int iters, uint32_t idesc, uint32_t* status)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (pk_smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sA = base, sB = base + 16384, bar = base + 16384 + 32768;
    __shared__ uint32_t s_tmem;
    // operands: arbitrary non-trivial bytes (small magnitudes; for bf16 the pattern gives finite values)
    for (uint32_t i = threadIdx.x; i < (16384 + 32768) / 4; i += blockDim.x) {
        uint32_t v = (i * 2654435761u) >> 7;
        v = is_bf16 ? (v & 0x007F007Fu) | 0x3C003C00u : (v & 0x0F0F0F0Fu);
        asm volatile("st.shared.b32 [%0], %1;" ::"r"(base + 4 * i), "r"(v) : "memory");
    }
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (threadIdx.x < 32) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 256;" ::"r"(pk_smem_u32(&s_tmem)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s_tmem;
    if (threadIdx.x == 0) {
        auto desc = [](uint32_t addr) {
            return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)1 << 16) | ((uint64_t)64 << 32) | ((uint64_t)1 << 46) |
                   ((uint64_t)2 << 61);
        };
        // The issuing thread must not be the limiter: the four descriptor pairs of a k-block are
        // formed once, and the loop over iterations holds nothing but the four instructions.
        uint64_t ad[4], bd[4];
        for (int ks = 0; ks < 4; ++ks) { ad[ks] = desc(sA) + 2 * ks; bd[ks] = desc(sB) + 2 * ks; }
        uint32_t phase = 0;
        bool ok = true;
        for (int it = 0; it < iters && ok; ++it) {
            // one "k-block": 4 instructions walking the 128-byte swizzle atom, like the layer kernel
            if (is_bf16) {
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                                 ::"r"(tmem), "l"(ad[ks]), "l"(bd[ks]), "r"(idesc), "r"(it | ks) : "memory");
            } else {
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                                 "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
                                 ::"r"(tmem), "l"(ad[ks]), "l"(bd[ks]), "r"(idesc), "r"(it | ks) : "memory");
            }
            if ((it & 7) == 7 || it == iters - 1) {
                asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
                // bounded wait for the batch
                const long long t0 = clock64();
                for (;;) {
                    uint32_t done;
                    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                                 "selp.u32 %0, 1, 0, p;\n\t}" : "=r"(done) : "r"(bar), "r"(phase) : "memory");
                    if (done) break;
                    if (clock64() - t0 > 2000000000LL) { ok = false; atomicMax(status, (uint32_t)RMSMP_ERR_TIMEOUT); break; }
                }
                phase ^= 1;
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x < 32) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 256;" ::"r"(tmem) : "memory");
    }
}

// One warp waits, with the kernels' own bounded wait, on an mbarrier that nobody ever arrives on.
// Nothing else is in flight (no bulk copy, no tensor-memory allocation), so giving up is all there is
// to do: the wait runs out after `limit_cycles`, the abort flag goes up, the status word receives
// RMSMP_ERR_TIMEOUT and the kernel returns normally.
__global__ void __launch_bounds__(32, 1) wait_expiry_kernel(long long limit_cycles, uint32_t* status)
{
    __shared__ uint64_t s_bar;
    __shared__ int s_abort;
    const uint32_t bar = smem_u32(&s_bar);
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    bool ok = true;
    if (threadIdx.x == 0) ok = mbar_wait(bar, 0, &s_abort, limit_cycles);
    ok = __all_sync(0xffffffffu, ok);
    if (threadIdx.x == 0 && !ok && s_abort) atomicMax(status, (uint32_t)RMSMP_ERR_TIMEOUT);
}

}  // namespace
}  // namespace rmsmp

extern "C" rmsmp_status rmsmp_selftest_bounded_wait(int64_t limit_cycles, uint32_t* d_status_word, void* stream)
{
    using namespace rmsmp;
    if (!d_status_word) return RMSMP_ERR_NULL;
    if (limit_cycles < 1 || limit_cycles > 200000000LL) return RMSMP_ERR_SHAPE;      // at most ~0.1 s
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
        cudaGetLastError();
        return RMSMP_ERR_CUDA;
    }
    if (major != 10) return RMSMP_ERR_ARCH;
    wait_expiry_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>((long long)limit_cycles, d_status_word);
    if (cudaGetLastError() != cudaSuccess) return RMSMP_ERR_CUDA;
    return RMSMP_OK;
}

extern "C" rmsmp_status rmsmp_measure_mma_peak(int use_bf16, int n_cols, int iters, uint32_t* d_status_word, float* h_tops, float* h_ms, void* stream)
{
    using namespace rmsmp;
    if (!h_tops || !d_status_word) return RMSMP_ERR_NULL;
    if (iters < 1 || iters > (1 << 22) || n_cols < 16 || n_cols > 256 || (n_cols & 15)) return RMSMP_ERR_SHAPE;
    int dev = 0, major = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
        cudaGetLastError();
        return RMSMP_ERR_CUDA;
    }
    if (major != 10) return RMSMP_ERR_ARCH;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint32_t* d_status = d_status_word;
    cudaEvent_t e0, e1;
    if (cudaMemsetAsync(d_status, 0, 4, st) != cudaSuccess) { cudaGetLastError(); return RMSMP_ERR_CUDA; }
    cudaFuncSetAttribute(mma_peak_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPeakSmem);
    // M=128 (bits 24-28 = 8), N/8 at bits 17-22; i8: s32 accumulate, signed A/B; bf16: f32 accumulate
    const uint32_t nfield = (uint32_t)(n_cols >> 3) << 17;
    const uint32_t idesc = use_bf16 ? ((1u << 4) | (1u << 7) | (1u << 10) | nfield | (8u << 24))
                                    : ((2u << 4) | (1u << 7) | (1u << 10) | nfield | (8u << 24));
    cudaEventCreate(&e0); cudaEventCreate(&e1);
    mma_peak_kernel<<<sms, kPeakThreads, kPeakSmem, st>>>(use_bf16, 64, idesc, d_status);   // warm-up
    cudaEventRecord(e0, st);
    mma_peak_kernel<<<sms, kPeakThreads, kPeakSmem, st>>>(use_bf16, iters, idesc, d_status);
    cudaEventRecord(e1, st);
    rmsmp_status rc = RMSMP_OK;
    float ms = 0.f;
    uint32_t hs = 0;
    if (cudaEventSynchronize(e1) != cudaSuccess || cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess ||
        cudaMemcpy(&hs, d_status, 4, cudaMemcpyDeviceToHost) != cudaSuccess) {
        cudaGetLastError();
        rc = RMSMP_ERR_CUDA;
    } else if (hs != 0) {
        rc = RMSMP_ERR_TIMEOUT;
    } else {
        const double k_per_instr = use_bf16 ? 16.0 : 32.0;
        const double ops = 2.0 * 128 * n_cols * k_per_instr * 4.0 * iters * sms;
        *h_tops = (float)(ops / (ms * 1e-3) / 1e12);
        if (h_ms) *h_ms = ms;
    }
    cudaEventDestroy(e0); cudaEventDestroy(e1);
    return rc;
}
