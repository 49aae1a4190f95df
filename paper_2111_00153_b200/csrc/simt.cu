// CUDA-core variants of the contraction: a one-thread-per-output cross-check kernel and a
// row-per-warp kernel (integer dot products on codes expanded in registers, or -- for PoT
// rows -- shifts and adds without a multiplier).
#include "common.cuh"
#include "decode.cuh"

namespace rmsmp {

__device__ __forceinline__ void store_result(const Problem& p, int64_t n, int m, int acc)
{
    const float c = __fmul_rn(p.wstep[m], p.act_step);
    const float y = __fmul_rn(__int2float_rn(acc), c);
    const int64_t o = p.out_mn ? (int64_t)m * p.ld_out + n : n * p.ld_out + m;
    p.out[o] = y;
    if (p.acc) p.acc[o] = acc;
}

// ------------------------------------------------------------------ one thread per output

__global__ void __launch_bounds__(256) simple_kernel(Problem p)
{
    const int64_t total = p.N * p.M;
    const int n4 = p.nP + p.nF4;
    for (int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; t < total;
         t += (int64_t)gridDim.x * blockDim.x) {
        const int m = (int)(t % p.M);
        const int64_t n = t / p.M;
        const int wo = (int)(n % p.Wo), ho = (int)((n / p.Wo) % p.Ho);
        const int64_t b = n / ((int64_t)p.Wo * p.Ho);
        const int kd = p.kind[m], ps = p.slot[m];
        const uint8_t* row4 = p.q4 + (size_t)ps * (p.Kp / 2);
        const int8_t* row8 = reinterpret_cast<const int8_t*>(p.q8) + (size_t)(ps - n4) * p.Kp;
        int acc = 0;
        for (int i = 0; i < p.kh; ++i) {
            const int y = ho * p.stride + i - p.pad;
            if (y < 0 || y >= p.H) continue;
            for (int j = 0; j < p.kw; ++j) {
                const int x = wo * p.stride + j - p.pad;
                if (x < 0 || x >= p.W) continue;
                const int8_t* a = p.act + ((b * p.H + y) * p.W + x) * p.pix_pitch;
                const int k0 = (i * p.kw + j) * p.Cp;
                for (int c = 0; c < p.Cin; ++c) {
                    const int v = (kd == kFixed8) ? (int)row8[k0 + c] : decode4(row4, k0 + c, kd);
                    acc += v * (int)a[c];
                }
            }
        }
        store_result(p, n, m, acc);
    }
}

cudaError_t launch_simple(const Problem& p, cudaStream_t st)
{
    int64_t total = p.N * p.M;
    int64_t blocks = (total + 255) / 256;
    if (blocks > 148 * 64) blocks = 148 * 64;
    simple_kernel<<<(unsigned)blocks, 256, 0, st>>>(p);
    return cudaGetLastError();
}

// ------------------------------------------------------------------ row per warp
// Work item = (packed row, group of kTok pixels).  Lanes stride over the 32-code chunks of
// the packed row (one coalesced 128-bit load per lane and step), expand them in registers
// and accumulate against the pixels' activation codes; a warp reduction finishes the sums.
// Consecutive warps take consecutive packed rows, so a warp's rows are of one kind.

constexpr int kTok = 8;

__device__ __forceinline__ int dot32(const uint32_t w[8], const uint32_t a[8], int acc)
{
#pragma unroll
    for (int q = 0; q < 8; ++q) acc = __dp4a((int)w[q], (int)a[q], acc);
    return acc;
}

// PoT row, multiplier-free: acc +-= a << (e-1) for each of the 32 codes of a packed chunk.
__device__ __forceinline__ int shiftadd32(const uint4& c, const uint32_t a[8], int acc)
{
    const uint32_t cw[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
    for (int w = 0; w < 4; ++w) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t nib = (cw[w] >> (4 * i)) & 15u;
            const int code = w * 8 + i;
            const int av = (int)(int8_t)((a[code >> 2] >> (8 * (code & 3))) & 0xFFu);
            const uint32_t e = nib & 7u;
            int term = (int)((uint32_t)av << ((e - 1u) & 7u));     // two's complement shift
            term = e ? term : 0;
            acc = (nib & 8u) ? acc - term : acc + term;
        }
    }
    return acc;
}

template <bool SHIFTADD>
__global__ void __launch_bounds__(256) rowwarp_kernel(Problem p)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int64_t ngroups = (p.N + kTok - 1) / kTok;
    const int32_t* perm = p.perm;
    const int n4 = p.nP + p.nF4;
    const int taps = p.kh * p.kw;
    const int nchunks = taps * (p.Cp >> 5);
    const bool vec_ok = ((p.pix_pitch & 15) == 0) && ((reinterpret_cast<uintptr_t>(p.act) & 15) == 0);

    for (int64_t work = warp; work < ngroups * p.M; work += nwarps) {
        const int pr = (int)(work % p.M);
        const int64_t n0 = (work / p.M) * kTok;
        const int m = perm[pr];
        const int kd = p.kind[m];
        const uint8_t* row = (kd == kFixed8) ? p.q8 + (size_t)(pr - n4) * p.Kp
                                             : p.q4 + (size_t)pr * (p.Kp / 2);
        // pixel coordinates of the group's tokens
        int y0[kTok], x0[kTok];
        int64_t bb[kTok];
#pragma unroll
        for (int t = 0; t < kTok; ++t) {
            int64_t n = n0 + t;
            if (n >= p.N) n = p.N - 1;
            x0[t] = (int)(n % p.Wo) * p.stride - p.pad;
            y0[t] = (int)((n / p.Wo) % p.Ho) * p.stride - p.pad;
            bb[t] = n / ((int64_t)p.Wo * p.Ho);
        }
        int acc[kTok];
#pragma unroll
        for (int t = 0; t < kTok; ++t) acc[t] = 0;

        for (int ch = lane; ch < nchunks; ch += 32) {
            const int kp = ch << 5;
            const int tap = kp / p.Cp, c0 = kp - tap * p.Cp;
            const int ti = tap / p.kw, tj = tap - ti * p.kw;
            uint32_t w[8];
            uint4 raw = make_uint4(0, 0, 0, 0);
            if (kd == kFixed8) {
                const uint4* src = reinterpret_cast<const uint4*>(row + kp);
                uint4 lo = __ldg(src), hi = __ldg(src + 1);
                w[0] = lo.x; w[1] = lo.y; w[2] = lo.z; w[3] = lo.w;
                w[4] = hi.x; w[5] = hi.y; w[6] = hi.z; w[7] = hi.w;
            } else {
                raw = __ldg(reinterpret_cast<const uint4*>(row + (kp >> 1)));
                if (kd == kPoT4) expand_pot_chunk(raw, w); else expand_fixed4_chunk_x16(raw, w);
            }
            const bool full = (c0 + 32 <= p.Cin) && vec_ok;
#pragma unroll
            for (int t = 0; t < kTok; ++t) {
                if (n0 + t >= p.N) break;
                const int y = y0[t] + ti, x = x0[t] + tj;
                if (y < 0 || y >= p.H || x < 0 || x >= p.W) continue;
                const int8_t* ap = p.act + ((bb[t] * p.H + y) * p.W + x) * p.pix_pitch + c0;
                uint32_t a[8];
                if (full) {
                    uint4 lo = __ldg(reinterpret_cast<const uint4*>(ap));
                    uint4 hi = __ldg(reinterpret_cast<const uint4*>(ap) + 1);
                    a[0] = lo.x; a[1] = lo.y; a[2] = lo.z; a[3] = lo.w;
                    a[4] = hi.x; a[5] = hi.y; a[6] = hi.z; a[7] = hi.w;
                } else {
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        uint32_t v = 0;
#pragma unroll
                        for (int bI = 0; bI < 4; ++bI) {
                            const int c = c0 + q * 4 + bI;
                            if (c < p.Cin) v |= (uint32_t)(uint8_t)ap[q * 4 + bI] << (8 * bI);
                        }
                        a[q] = v;
                    }
                }
                if (SHIFTADD && kd == kPoT4) acc[t] = shiftadd32(raw, a, acc[t]);
                else acc[t] = dot32(w, a, acc[t]);
            }
        }
#pragma unroll
        for (int t = 0; t < kTok; ++t) {
            int v = acc[t];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            if (kd == kFixed4) v >>= 4;   // the Fixed-4 codes were expanded as 16 * value
            if (lane == t && n0 + t < p.N) store_result(p, n0 + t, m, v);
        }
    }
}

cudaError_t launch_simt(const Problem& p, bool shiftadd, cudaStream_t st)
{
    const int64_t ngroups = (p.N + kTok - 1) / kTok;
    int64_t warps = ngroups * p.M;
    int64_t blocks = (warps + 7) / 8;
    if (blocks > 148 * 8) blocks = 148 * 8;
    if (shiftadd) rowwarp_kernel<true><<<(unsigned)blocks, 256, 0, st>>>(p);
    else rowwarp_kernel<false><<<(unsigned)blocks, 256, 0, st>>>(p);
    return cudaGetLastError();
}

}  // namespace rmsmp
