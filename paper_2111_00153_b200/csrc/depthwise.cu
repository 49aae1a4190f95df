// Depthwise convolution (one input channel per filter, as in MobileNet-v2's 3x3 layers): every channel c
// has its own filter row with its own scheme and precision (Figure 2), y[b][ho][wo][c] = sum over the
// taps of value[c][i][j] * a[b][ho*s+i-p][wo*s+j-p][c].  There is no reduction over channels, hence no
// matrix product: the layer is bound by its output write, and the work is one integer multiply-add per
// tap on the CUDA cores.  A block expands the layer's codes once into shared memory, four channels per
// word and one word per channel of the quad with the other three bytes zero, so that a 4-way byte dot
// product of the activation word of a channel quad with that word is exactly one channel's product.
#include "common.cuh"

namespace rmsmp {

namespace {

constexpr int kDwThreads = 256;

__global__ void __launch_bounds__(kDwThreads) depthwise_kernel(const Problem p)
{
    extern __shared__ uint32_t s_w[];                     // [tap][channel]: the channel's value in byte (channel & 3)
    const int taps = p.kh * p.kw, C = p.M;
    for (int i = threadIdx.x; i < taps * C; i += kDwThreads) {
        const int tap = i / C, c = i - tap * C;
        const int kind = p.kind[c], slot = p.slot[c];
        int v;
        if (kind == kFixed8) v = (int)(int8_t)p.q8[(size_t)(slot - p.nP - p.nF4) * p.Kp + tap * p.Cp];
        else v = decode4(p.q4 + (size_t)slot * (p.Kp >> 1), tap * p.Cp, kind);
        s_w[i] = (uint32_t)(v & 0xFF) << (8 * (c & 3));
    }
    __syncthreads();
    const int quads = C >> 2;
    const int64_t work = p.N * quads;                     // (output pixel, channel quad)
    for (int64_t w = blockIdx.x * (int64_t)kDwThreads + threadIdx.x; w < work; w += (int64_t)gridDim.x * kDwThreads) {
        const int64_t n = w / quads;
        const int q = (int)(w - n * quads);
        const int wo = (int)(n % p.Wo), ho = (int)((n / p.Wo) % p.Ho);
        const int64_t b = n / ((int64_t)p.Wo * p.Ho);
        int acc[4] = {0, 0, 0, 0};
        for (int i = 0; i < p.kh; ++i) {
            const int y = ho * p.stride + i - p.pad;
            if (y < 0 || y >= p.H) continue;
            for (int j = 0; j < p.kw; ++j) {
                const int x = wo * p.stride + j - p.pad;
                if (x < 0 || x >= p.W) continue;
                const uint32_t a4 = __ldg(reinterpret_cast<const uint32_t*>(p.act + ((b * p.H + y) * p.W + x) * p.pix_pitch) + q);
                const uint4 w4 = *reinterpret_cast<const uint4*>(s_w + (i * p.kw + j) * C + 4 * q);
                acc[0] = __dp4a((int)a4, (int)w4.x, acc[0]);
                acc[1] = __dp4a((int)a4, (int)w4.y, acc[1]);
                acc[2] = __dp4a((int)a4, (int)w4.z, acc[2]);
                acc[3] = __dp4a((int)a4, (int)w4.w, acc[3]);
            }
        }
        const float4 ws = __ldg(reinterpret_cast<const float4*>(p.wstep) + q);
        float4 o;
        o.x = __fmul_rn(__int2float_rn(acc[0]), __fmul_rn(ws.x, p.act_step));
        o.y = __fmul_rn(__int2float_rn(acc[1]), __fmul_rn(ws.y, p.act_step));
        o.z = __fmul_rn(__int2float_rn(acc[2]), __fmul_rn(ws.z, p.act_step));
        o.w = __fmul_rn(__int2float_rn(acc[3]), __fmul_rn(ws.w, p.act_step));
        reinterpret_cast<float4*>(p.out + n * p.ld_out)[q] = o;
        if (p.acc) reinterpret_cast<int4*>(p.acc + n * p.ld_out)[q] = make_int4(acc[0], acc[1], acc[2], acc[3]);
    }
}

}  // namespace

// Channels a multiple of 4, the expanded filter table within shared memory.
bool depthwise_supported(const Problem& p)
{
    return p.Cin == 1 && (p.M & 3) == 0 && (size_t)p.kh * p.kw * p.M * 4 <= 200 * 1024 && (p.pix_pitch & 3) == 0 && (p.ld_out & 3) == 0;
}

cudaError_t launch_depthwise(const Problem& p, cudaStream_t st)
{
    const size_t smem = (size_t)p.kh * p.kw * p.M * 4;
    static bool attr_set[kMaxDevices] = {};
    if (smem > 48 * 1024 && !ensure_smem_attr(reinterpret_cast<const void*>(depthwise_kernel), 200 * 1024, attr_set)) return cudaErrorUnknown;
    const int64_t work = p.N * (p.M >> 2);
    int64_t blocks = (work + kDwThreads - 1) / kDwThreads;
    const int64_t cap = (int64_t)sm_count() * (smem > 64 * 1024 ? 1 : 4);
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    depthwise_kernel<<<(unsigned)blocks, kDwThreads, smem, st>>>(p);
    return cudaGetLastError();
}

}  // namespace rmsmp
