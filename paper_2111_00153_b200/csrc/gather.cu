// Patch matrix of a convolution's activation codes, for layers whose channel count is too small for the
// implicit form (a network's first layer: 3 channels, 7 x 7 filters; Section 4.1, Table 6 quantizes it like
// the rest): cols[n][(i * kw + j) * C + c] = act[b][ho * s + i - p][wo * s + j - p][c] for output pixel
// n = (b, ho, wo), zero outside the image and in the columns beyond kh * kw * C.  The layer is then a linear
// layer over these rows (reduction order tap-major, channel fastest), which the GEMM entry points take.
// A filter tap of such a layer is 3 bytes, which no bulk tensor copy can start on (16-byte rule), so this is
// plain loads: the input is read many times, but it is small and stays in L1/L2; the kernel is bound by
// writing the matrix.  One thread per 16 output bytes, stepping through filter row, column and channel.
#include <algorithm>
#include "common.cuh"

namespace rmsmp {

namespace {

constexpr int kGatherThreads = 256;

struct GatherArgs {
    const int8_t* act;
    int8_t* cols;
    int64_t pix_pitch, ld_cols, N;
    int B, H, W, C, kh, kw, stride, pad, Ho, Wo, K, units;      // units: 16-byte pieces per output row
};

__global__ void __launch_bounds__(kGatherThreads) im2col_kernel(const GatherArgs a)
{
    // thread <-> (pixel of the block's current group, 16-byte piece of its row): fixed per thread; the pixel index
    // advances by whole groups; 32-bit index arithmetic (the host checks the counts)
    const int upr = a.units;
    const int ppg = kGatherThreads / upr;                 // pixels per group (units <= kGatherThreads is checked by the host)
    const int my_p = threadIdx.x / upr, k0 = (threadIdx.x - my_p * upr) << 4;
    if (my_p >= ppg) return;
    const int tap0 = k0 / a.C, c0 = k0 - tap0 * a.C;
    const int i0 = tap0 / a.kw, j0 = tap0 - i0 * a.kw;
    const uint32_t N = (uint32_t)a.N;
    const int64_t row_pitch = (int64_t)a.W * a.pix_pitch;
    for (uint32_t n = blockIdx.x * (uint32_t)ppg + my_p; n < N; n += gridDim.x * (uint32_t)ppg) {
        const uint32_t t = n / (uint32_t)a.Wo;
        const int wo = (int)(n - t * (uint32_t)a.Wo);
        const uint32_t b = t / (uint32_t)a.Ho;
        const int ho = (int)(t - b * (uint32_t)a.Ho);
        const int y0 = ho * a.stride - a.pad, x0 = wo * a.stride - a.pad;
        int i = i0, j = j0, c = c0;
        const int8_t* ptr = a.act + (int64_t)b * a.H * row_pitch + (int64_t)(y0 + i) * row_pitch + (int64_t)(x0 + j) * a.pix_pitch + c;
        bool yok = (unsigned)(y0 + i) < (unsigned)a.H;
        uint32_t out[4] = {0u, 0u, 0u, 0u};
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            if (k0 + e < a.K) {
                if (yok && (unsigned)(x0 + j) < (unsigned)a.W) out[e >> 2] |= (uint32_t)(uint8_t)__ldg(ptr) << (8 * (e & 3));
                ++ptr;
                if (++c == a.C) {
                    c = 0;
                    ptr += a.pix_pitch - a.C;
                    if (++j == a.kw) {
                        j = 0; ++i;
                        ptr += row_pitch - (int64_t)a.kw * a.pix_pitch;
                        yok = (unsigned)(y0 + i) < (unsigned)a.H;
                    }
                }
            }
        }
        *reinterpret_cast<uint4*>(a.cols + (int64_t)n * a.ld_cols + k0) = make_uint4(out[0], out[1], out[2], out[3]);
    }
}

// The same through shared memory, one output row (b, ho) per block pass: the kh input rows it touches are copied
// in first, channels packed and the horizontal padding as zeros, so that a thread's 16 source offsets are fixed
// for all pixels of all rows and its loop has no bounds checks.  s_rows[kh][rowb].
__global__ void __launch_bounds__(kGatherThreads) im2col_rows_kernel(const GatherArgs a, const int Wx, const int rowb)
{
    extern __shared__ uint8_t s_rows[];
    const int upr = a.units;
    const int ppg = kGatherThreads / upr;
    const int my_p = threadIdx.x / upr, k0 = (threadIdx.x - my_p * upr) << 4;
    int off[16];
    uint32_t keep[4] = {0u, 0u, 0u, 0u};                  // byte masks: columns beyond the reduction stay zero
#pragma unroll
    for (int e = 0; e < 16; ++e) {
        const int k = k0 + e;
        const int tap = k / a.C, c = k - tap * a.C;
        const int i = tap / a.kw, j = tap - i * a.kw;
        const bool valid = k < a.K;
        off[e] = valid ? i * rowb + j * a.C + c : 0;      // offsets are relative to the pixel's first byte: 0 is always inside
        if (valid) keep[e >> 2] |= 0xFFu << (8 * (e & 3));
    }
    const int64_t row_pitch = (int64_t)a.W * a.pix_pitch;
    const int rows_total = a.B * a.Ho;
    for (int r = blockIdx.x; r < rows_total; r += gridDim.x) {
        const int b = r / a.Ho, ho = r - b * a.Ho;
        const int y0 = ho * a.stride - a.pad;
        __syncthreads();                                  // the previous row's readers are done
        for (int q = threadIdx.x; q < a.kh * Wx; q += kGatherThreads) {
            const int i = q / Wx, xp = q - i * Wx;
            const int y = y0 + i, x = xp - a.pad;
            const bool in = (unsigned)y < (unsigned)a.H && (unsigned)x < (unsigned)a.W;
            const int8_t* src = a.act + (int64_t)b * a.H * row_pitch + (int64_t)y * row_pitch + (int64_t)x * a.pix_pitch;
            uint8_t* dst = s_rows + i * rowb + xp * a.C;
            for (int c = 0; c < a.C; ++c) dst[c] = in ? (uint8_t)__ldg(src + c) : (uint8_t)0;
        }
        __syncthreads();
        if (my_p < ppg) {
            for (int wo = my_p; wo < a.Wo; wo += ppg) {
                const uint8_t* base = s_rows + wo * a.stride * a.C;
                uint32_t out[4] = {0u, 0u, 0u, 0u};
#pragma unroll
                for (int e = 0; e < 16; ++e) out[e >> 2] |= (uint32_t)base[off[e]] << (8 * (e & 3));
                *reinterpret_cast<uint4*>(a.cols + ((int64_t)r * a.Wo + wo) * a.ld_cols + k0) =
                    make_uint4(out[0] & keep[0], out[1] & keep[1], out[2] & keep[2], out[3] & keep[3]);
            }
        }
    }
}

}  // namespace

cudaError_t launch_im2col(const int8_t* act, int B, int H, int W, int C, int64_t pix_pitch, int kh, int kw, int stride, int pad,
                          int Ho, int Wo, int8_t* cols, int64_t ld_cols, cudaStream_t st)
{
    GatherArgs a;
    a.act = act; a.cols = cols; a.pix_pitch = pix_pitch; a.ld_cols = ld_cols;
    a.B = B; a.H = H; a.W = W; a.C = C; a.kh = kh; a.kw = kw; a.stride = stride; a.pad = pad; a.Ho = Ho; a.Wo = Wo;
    a.N = (int64_t)B * Ho * Wo;
    a.K = kh * kw * C;
    a.units = (int)(ld_cols >> 4);
    if (a.N == 0) return cudaSuccess;
    if (a.units > kGatherThreads) return cudaErrorInvalidValue;
    // input rows in shared memory when they fit without opting in to more
    const int Wx = (Wo - 1) * stride + kw;
    const int rowb = (Wx * C + 15) & ~15;
    const size_t smem = (size_t)kh * rowb + 16;
    if (smem <= 48 * 1024) {
        const int64_t blocks = std::min<int64_t>((int64_t)B * Ho, (int64_t)sm_count() * 8);
        im2col_rows_kernel<<<(unsigned)blocks, kGatherThreads, smem, st>>>(a, Wx, rowb);
        return cudaGetLastError();
    }
    const int ppg = kGatherThreads / a.units;
    const int64_t blocks = std::min<int64_t>((a.N + ppg - 1) / ppg, (int64_t)sm_count() * 16);
    im2col_kernel<<<(unsigned)blocks, kGatherThreads, 0, st>>>(a);
    return cudaGetLastError();
}

}  // namespace rmsmp
