// Depthwise convolution (one input channel per filter, as in MobileNet-v2's 3x3 layers): every channel c
// has its own filter row with its own scheme and precision (Figure 2), y[b][ho][wo][c] = sum over the
// taps of value[c][i][j] * a[b][ho*s+i-p][wo*s+j-p][c].  There is no reduction over channels, hence no
// matrix product: the layer is bound by its output write, and the work is one integer multiply-add per
// tap on the CUDA cores.  A block expands the layer's codes once into shared memory, one word per tap and
// channel quad (channel 4q+j in byte j).  An activation word of a quad is split into four words that keep
// one channel's byte each, and a 4-way byte dot product of such a word with the weight word is exactly
// that channel's product.  For 3 x 3 filters of stride 1 or 2 a thread owns one quad, keeps its nine
// weight words in registers and computes a run of four neighbouring outputs of a row, so that every
// loaded and split activation word serves all the taps that touch it.
#include <algorithm>
#include "common.cuh"

namespace rmsmp {

namespace {

constexpr int kDwThreads = 256;
constexpr int kDwRun = 4;                                  // outputs of one row per thread (3 x 3 path)

__device__ __forceinline__ void dw_store(const Problem& p, uint32_t n, int q, const int* acc)
{
    const float4 ws = __ldg(reinterpret_cast<const float4*>(p.wstep) + q);
    float4 o;
    o.x = __fmul_rn(__int2float_rn(acc[0]), __fmul_rn(ws.x, p.act_step));
    o.y = __fmul_rn(__int2float_rn(acc[1]), __fmul_rn(ws.y, p.act_step));
    o.z = __fmul_rn(__int2float_rn(acc[2]), __fmul_rn(ws.z, p.act_step));
    o.w = __fmul_rn(__int2float_rn(acc[3]), __fmul_rn(ws.w, p.act_step));
    reinterpret_cast<float4*>(p.out + (size_t)n * p.ld_out)[q] = o;
    if (p.acc) reinterpret_cast<int4*>(p.acc + (size_t)n * p.ld_out)[q] = make_int4(acc[0], acc[1], acc[2], acc[3]);
}

// kS = 1, 2: 3 x 3 filters of that stride, runs of kDwRun outputs; kS = 0: any filter, one output per item.
template <int kS>
__global__ void __launch_bounds__(kDwThreads, 4) depthwise_kernel(const Problem p)
{
    extern __shared__ uint32_t s_w[];                     // [tap][quad]: channel 4q+j in byte j
    const int taps = p.kh * p.kw, C = p.M;
    {
        uint8_t* s_b = reinterpret_cast<uint8_t*>(s_w);
        for (int c = threadIdx.x; c < C; c += kDwThreads) {
            const int kind = p.kind[c], slot = p.slot[c];
            const uint8_t* r8 = p.q8 + (kind == kFixed8 ? (size_t)(slot - p.nP - p.nF4) * p.Kp : 0);
            const uint8_t* r4 = p.q4 + (size_t)slot * (p.Kp >> 1);
            for (int tap = 0; tap < taps; ++tap)
                s_b[tap * C + c] = (uint8_t)(kind == kFixed8 ? (int)(int8_t)r8[tap * p.Cp] : decode4(r4, tap * p.Cp, kind));
        }
    }
    __syncthreads();
    const int quads = C >> 2;
    // thread <-> (item of the block's current group, channel quad): the split is fixed per thread, the item
    // index advances by whole groups, and all index arithmetic is 32-bit (the host checks the counts)
    const int qpt = (quads + kDwThreads - 1) / kDwThreads;             // quads per thread when an item has more quads than threads
    const int lanes_q = min(quads, kDwThreads);                        // threads that share an item
    const int ipg = kDwThreads / lanes_q;                              // items per group
    const int my_i = threadIdx.x / lanes_q, my_q0 = threadIdx.x - my_i * lanes_q;
    if (my_i >= ipg) return;
    if constexpr (kS != 0) {
        const uint32_t rpr = (uint32_t)(p.Wo + kDwRun - 1) / kDwRun;   // runs per output row
        const uint32_t n_runs = (uint32_t)(p.N / p.Wo) * rpr;
        constexpr int kXW = (kDwRun - 1) * kS + 3;                     // input columns a run touches
        for (int qi = 0; qi < qpt; ++qi) {
            const int q = my_q0 + qi * lanes_q;
            if (q >= quads) break;
            uint32_t w9[9];
#pragma unroll
            for (int t = 0; t < 9; ++t) w9[t] = s_w[t * quads + q];
            for (uint32_t run = blockIdx.x * (uint32_t)ipg + my_i; run < n_runs; run += gridDim.x * (uint32_t)ipg) {
                const uint32_t bh = run / rpr;                         // image * Ho + output row
                const int wo0 = (int)(run - bh * rpr) * kDwRun;
                const uint32_t b = bh / (uint32_t)p.Ho;
                const int ho = (int)(bh - b * (uint32_t)p.Ho);
                const int8_t* img = p.act + (size_t)b * p.H * p.W * p.pix_pitch;
                int acc[kDwRun][4];
#pragma unroll
                for (int r = 0; r < kDwRun; ++r) acc[r][0] = acc[r][1] = acc[r][2] = acc[r][3] = 0;
                // all loads of the run first (rows and columns outside the image read as zero), then the arithmetic
                uint32_t a[3][kXW];
#pragma unroll
                for (int i = 0; i < 3; ++i) {
                    const int y = ho * kS + i - p.pad;
                    const bool yin = y >= 0 && y < p.H;
                    const int8_t* rowp = img + (size_t)(yin ? y : 0) * p.W * p.pix_pitch;
#pragma unroll
                    for (int xx = 0; xx < kXW; ++xx) {
                        const int x = wo0 * kS + xx - p.pad;
                        a[i][xx] = (yin && x >= 0 && x < p.W) ? __ldg(reinterpret_cast<const uint32_t*>(rowp + (size_t)x * p.pix_pitch) + q) : 0u;
                    }
                }
#pragma unroll
                for (int i = 0; i < 3; ++i) {
#pragma unroll
                    for (int xx = 0; xx < kXW; ++xx) {
                        const int a0 = (int)(a[i][xx] & 0x000000FFu), a1 = (int)(a[i][xx] & 0x0000FF00u);
                        const int a2 = (int)(a[i][xx] & 0x00FF0000u), a3 = (int)(a[i][xx] & 0xFF000000u);
#pragma unroll
                        for (int j = 0; j < 3; ++j) {
                            if ((xx - j) % kS != 0 || xx - j < 0 || (xx - j) / kS >= kDwRun) continue;
                            const int r = (xx - j) / kS;
                            const int w = (int)w9[i * 3 + j];
                            acc[r][0] = __dp4a(a0, w, acc[r][0]);
                            acc[r][1] = __dp4a(a1, w, acc[r][1]);
                            acc[r][2] = __dp4a(a2, w, acc[r][2]);
                            acc[r][3] = __dp4a(a3, w, acc[r][3]);
                        }
                    }
                }
#pragma unroll
                for (int r = 0; r < kDwRun; ++r)
                    if (wo0 + r < p.Wo) dw_store(p, bh * (uint32_t)p.Wo + (uint32_t)(wo0 + r), q, acc[r]);
            }
        }
        return;
    } else {
    const uint32_t N = (uint32_t)p.N, hw = (uint32_t)(p.Ho * p.Wo);
    for (uint32_t n = blockIdx.x * (uint32_t)ipg + my_i; n < N; n += gridDim.x * (uint32_t)ipg) {
        const uint32_t b = n / hw, r = n - b * hw;
        const int ho = (int)(r / (uint32_t)p.Wo), wo = (int)(r - (uint32_t)ho * p.Wo);
        const int8_t* img = p.act + (size_t)b * p.H * p.W * p.pix_pitch;
        for (int qi = 0; qi < qpt; ++qi) {
            const int q = my_q0 + qi * lanes_q;
            if (q >= quads) break;
            int acc[4] = {0, 0, 0, 0};
            for (int i = 0; i < p.kh; ++i) {
                const int y = ho * p.stride + i - p.pad;
                if (y < 0 || y >= p.H) continue;
                for (int j = 0; j < p.kw; ++j) {
                    const int x = wo * p.stride + j - p.pad;
                    if (x < 0 || x >= p.W) continue;
                    const uint32_t a4 = __ldg(reinterpret_cast<const uint32_t*>(img + (size_t)(y * p.W + x) * p.pix_pitch) + q);
                    const int w = (int)s_w[(i * p.kw + j) * quads + q];
                    acc[0] = __dp4a((int)(a4 & 0x000000FFu), w, acc[0]);
                    acc[1] = __dp4a((int)(a4 & 0x0000FF00u), w, acc[1]);
                    acc[2] = __dp4a((int)(a4 & 0x00FF0000u), w, acc[2]);
                    acc[3] = __dp4a((int)(a4 & 0xFF000000u), w, acc[3]);
                }
            }
            dw_store(p, n, q, acc);
        }
    }
    }
}

}  // namespace

// Channels a multiple of 4, the expanded filter table within shared memory, 32-bit pixel counts.
bool depthwise_supported(const Problem& p)
{
    return p.Cin == 1 && (p.M & 3) == 0 && (size_t)p.kh * p.kw * p.M <= 200 * 1024 && (p.pix_pitch & 3) == 0 && (p.ld_out & 3) == 0 &&
           p.N < (int64_t)1 << 31;
}

cudaError_t launch_depthwise(const Problem& p, cudaStream_t st)
{
    const size_t smem = (size_t)p.kh * p.kw * p.M;
    const int variant = (p.kh == 3 && p.kw == 3 && (p.stride == 1 || p.stride == 2)) ? p.stride : 0;
    static bool attr_set[3][kMaxDevices] = {};
    const void* fn = variant == 1 ? reinterpret_cast<const void*>(depthwise_kernel<1>)
                   : variant == 2 ? reinterpret_cast<const void*>(depthwise_kernel<2>)
                                  : reinterpret_cast<const void*>(depthwise_kernel<0>);
    if (smem > 48 * 1024 && !ensure_smem_attr(fn, 200 * 1024, attr_set[variant])) return cudaErrorUnknown;
    int per_sm = 0;
    cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, kDwThreads, smem);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) per_sm = 1;
    const int quads = p.M >> 2;
    const int ipg = kDwThreads / std::min(quads, kDwThreads);          // items a block takes per pass
    const int64_t items = variant ? (p.N / p.Wo) * ((p.Wo + kDwRun - 1) / kDwRun) : p.N;
    // at least four passes per block, so that expanding the filter table stays a small part of its work
    int64_t blocks = ((items + ipg - 1) / ipg + 3) / 4;
    const int64_t cap = (int64_t)sm_count() * per_sm;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    if (variant == 1) depthwise_kernel<1><<<(unsigned)blocks, kDwThreads, smem, st>>>(p);
    else if (variant == 2) depthwise_kernel<2><<<(unsigned)blocks, kDwThreads, smem, st>>>(p);
    else depthwise_kernel<0><<<(unsigned)blocks, kDwThreads, smem, st>>>(p);
    return cudaGetLastError();
}

}  // namespace rmsmp
