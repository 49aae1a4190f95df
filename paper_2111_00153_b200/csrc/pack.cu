// Weight quantize + group + pack, its inverse (parity/debug), and the activation quantizer.
#include "common.cuh"
#include "decode.cuh"
#include "actq.cuh"

namespace rmsmp {

// ------------------------------------------------------------------ quantizers (fp32, one
// IEEE operation per step; intrinsics keep the compiler from fusing multiply and add)

__device__ __forceinline__ float clip_unit(float w, float alpha)   // Eq. 3
{
    float t = __fdiv_rn(w, alpha);
    t = fmaxf(t, -1.0f);
    t = fminf(t, 1.0f);
    return t;
}

__device__ __forceinline__ int fixed_q(float w, float alpha, float Q)   // Eq. 1-2
{
    return __float2int_rn(__fmul_rn(clip_unit(w, alpha), Q));
}

__device__ __forceinline__ int pot_nibble(float w, float alpha, int mode)   // Eq. 4-5
{
    float t = clip_unit(w, alpha);
    int s = (t < 0.0f) ? 8 : 0;
    float x = fabsf(t);
    int e = 0;
    if (mode == RMSMP_POT_NEAREST) {
        // midpoints between neighbouring levels; a value on a midpoint takes the larger level
        e = (x >= 0.0078125f) ? 1 : 0;      // 2^-7
        e = (x >= 0.0234375f) ? 2 : e;      // 3*2^-7
        e = (x >= 0.046875f) ? 3 : e;       // 3*2^-6
        e = (x >= 0.09375f) ? 4 : e;        // 3*2^-5
        e = (x >= 0.1875f) ? 5 : e;         // 3*2^-4
        e = (x >= 0.375f) ? 6 : e;          // 3*2^-3
        e = (x >= 0.75f) ? 7 : e;           // 3*2^-2
    } else {
        // round(log2 x) = j-7  <=>  x^2 >= 2^(2(j-7)-1); x^2 is exact in double
        double xx = (double)x * (double)x;
        double bound = 1.0 / 8192.0;        // 2^-13
#pragma unroll
        for (int k = 1; k <= 7; ++k) {
            e = (xx >= bound) ? k : e;
            bound *= 4.0;
        }
    }
    return e ? (s | e) : 0;
}

// ------------------------------------------------------------------ pack kernel
// One block per packed row.  Phase 1: coalesced (128-bit where aligned) reads of the fp32 row,
// quantize, scatter the codes as bytes into shared memory at their packed position k'.
// Phase 2: every thread turns 32 code bytes into one 16-byte (4-bit rows) or two 16-byte
// (8-bit rows) chunks and stores them with 128-bit stores, consecutive threads to consecutive
// chunks.

struct PackArgs {
    const float* W;
    uint8_t* blob;
    uint64_t off_perm, off_alpha, off_kind, off_q4, off_q8;
    int M, K, taps, Cin, Cp, Kp, n4, seg;   // seg: codes per shared-memory segment
    int conv, pot_mode;
};

__global__ void __launch_bounds__(256) pack_kernel(PackArgs a)
{
    extern __shared__ __align__(16) uint8_t s_code[];
    const int p = blockIdx.x;
    const int r = reinterpret_cast<const int32_t*>(a.blob + a.off_perm)[p];
    const float alpha = reinterpret_cast<const float*>(a.blob + a.off_alpha)[r];
    const int kind = (a.blob + a.off_kind)[r];
    const float* wrow = a.W + (size_t)r * a.K;
    const float Q = (kind == kFixed8) ? 127.0f : 7.0f;
    uint8_t* dst = (kind == kFixed8) ? a.blob + a.off_q8 + (size_t)(p - a.n4) * a.Kp
                                     : a.blob + a.off_q4 + (size_t)p * (a.Kp / 2);
    const bool vec4 = ((a.K & 3) == 0);   // row starts stay 16-byte aligned

    for (int seg0 = 0; seg0 < a.Kp; seg0 += a.seg) {
        const int seg_len = min(a.seg, a.Kp - seg0);
        for (int i = threadIdx.x * 16; i < seg_len; i += blockDim.x * 16)
            *reinterpret_cast<uint4*>(s_code + i) = make_uint4(0, 0, 0, 0);
        __syncthreads();
        // original indices covered by this segment (linear: k' = k; conv: whole row in one segment)
        const int k_lo = a.conv ? 0 : seg0;
        const int k_hi = a.conv ? a.K : min(a.K, seg0 + seg_len);
        auto put = [&](int idx, float w) {
            int code = (kind == kPoT4) ? pot_nibble(w, alpha, a.pot_mode) : fixed_q(w, alpha, Q);
            int kp = a.conv ? ((idx % a.taps) * a.Cp + idx / a.taps) : idx;
            s_code[kp - seg0] = (uint8_t)code;
        };
        if (vec4) {
            // four 128-bit loads in flight per thread before any code is formed: a block walks one
            // row, so its time is the number of dependent load rounds
            const int stride = blockDim.x * 4;
            for (int idx0 = k_lo + threadIdx.x * 4; idx0 < k_hi; idx0 += 4 * stride) {
                float4 w[4];
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (idx0 + u * stride < k_hi) w[u] = __ldg(reinterpret_cast<const float4*>(wrow + idx0 + u * stride));
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int idx = idx0 + u * stride;
                    if (idx < k_hi) { put(idx, w[u].x); put(idx + 1, w[u].y); put(idx + 2, w[u].z); put(idx + 3, w[u].w); }
                }
            }
        } else {
            for (int idx = k_lo + threadIdx.x; idx < k_hi; idx += blockDim.x) put(idx, wrow[idx]);
        }
        __syncthreads();
        for (int c = threadIdx.x; c < seg_len / 32; c += blockDim.x) {
            uint4 lo = *reinterpret_cast<const uint4*>(s_code + c * 32);
            uint4 hi = *reinterpret_cast<const uint4*>(s_code + c * 32 + 16);
            if (kind == kFixed8) {
                uint4* o = reinterpret_cast<uint4*>(dst + seg0 + c * 32);
                o[0] = lo; o[1] = hi;
            } else {
                const uint32_t l[4] = {lo.x, lo.y, lo.z, lo.w}, h[4] = {hi.x, hi.y, hi.z, hi.w};
                uint32_t o[4];
                if (kind == kFixed4) {
                    // byte b = code[b] << 4 | code[16+b]
#pragma unroll
                    for (int w = 0; w < 4; ++w) o[w] = ((l[w] << 4) & 0xF0F0F0F0u) | (h[w] & 0x0F0F0F0Fu);
                } else {
                    // byte b = code[2b] | code[2b+1] << 4
                    const uint32_t all[8] = {l[0], l[1], l[2], l[3], h[0], h[1], h[2], h[3]};
#pragma unroll
                    for (int w = 0; w < 4; ++w) {
                        uint32_t a0 = all[2 * w], a1 = all[2 * w + 1];   // codes 8w..8w+3, 8w+4..8w+7
                        uint32_t b0 = (a0 & 0xF) | ((a0 >> 4) & 0xF0);               // codes 0,1
                        uint32_t b1 = ((a0 >> 16) & 0xF) | ((a0 >> 20) & 0xF0);      // codes 2,3
                        uint32_t b2 = (a1 & 0xF) | ((a1 >> 4) & 0xF0);
                        uint32_t b3 = ((a1 >> 16) & 0xF) | ((a1 >> 20) & 0xF0);
                        o[w] = b0 | (b1 << 8) | (b2 << 16) | (b3 << 24);
                    }
                }
                *reinterpret_cast<uint4*>(dst + (seg0 + c * 32) / 2) = make_uint4(o[0], o[1], o[2], o[3]);
            }
        }
        __syncthreads();
    }
}

cudaError_t launch_pack(const float* dW, int conv_oihw, const rmsmp_layer& L, int pot_mode,
                        uint8_t* blob, cudaStream_t st)
{
    PackArgs a;
    a.W = dW; a.blob = blob;
    a.off_perm = L.off_perm; a.off_alpha = L.off_alpha; a.off_kind = L.off_kind;
    a.off_q4 = L.off_q4; a.off_q8 = L.off_q8;
    a.M = L.M; a.K = L.Cin * L.kh * L.kw; a.taps = L.kh * L.kw; a.Cin = L.Cin; a.Cp = L.Cp;
    a.Kp = L.Kp; a.n4 = L.nP + L.nF4;
    a.conv = (conv_oihw && a.taps > 1) ? 1 : 0;
    a.pot_mode = pot_mode;
    a.seg = a.conv ? L.Kp : (L.Kp < 32768 ? L.Kp : 32768);
    size_t smem = (size_t)a.seg;
    if (smem > 48 * 1024) {            // rows longer than the default dynamic shared memory limit
        cudaError_t e = cudaFuncSetAttribute(pack_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    pack_kernel<<<L.M, 256, smem, st>>>(a);
    return cudaGetLastError();
}

// ------------------------------------------------------------------ metadata fetch
// The few KB of per-row metadata come from mapped pinned host memory: 128-bit reads across the
// host link, 128-bit writes to the packed buffer.

__global__ void __launch_bounds__(256) fetch_mapped_kernel(uint8_t* __restrict__ dst, const uint8_t* __restrict__ src,
                                                           size_t bytes)
{
    const size_t n16 = bytes / 16;
    const size_t tid = blockIdx.x * (size_t)blockDim.x + threadIdx.x, nthr = (size_t)gridDim.x * blockDim.x;
    // host memory: loads that bypass the caches, so that a reused slot is never read stale
    for (size_t i = tid; i < n16; i += nthr)
        reinterpret_cast<uint4*>(dst)[i] = __ldcv(reinterpret_cast<const uint4*>(src) + i);
    for (size_t i = n16 * 16 + tid; i < bytes; i += nthr) dst[i] = __ldcv(src + i);
}

cudaError_t launch_fetch_mapped(void* d_dst, const void* mapped_src, size_t bytes, cudaStream_t st)
{
    size_t blocks = (bytes / 16 + 255) / 256;
    if (blocks > 64) blocks = 64;
    if (blocks == 0) blocks = 1;
    fetch_mapped_kernel<<<(unsigned)blocks, 256, 0, st>>>(static_cast<uint8_t*>(d_dst), static_cast<const uint8_t*>(mapped_src), bytes);
    return cudaGetLastError();
}

// ------------------------------------------------------------------ unpack (parity/debug)

__global__ void unpack_kernel(const uint8_t* blob, rmsmp_layer L, int8_t* values, int32_t* perm,
                              float* wstep)
{
    const int K = L.Cin * L.kh * L.kw, taps = L.kh * L.kw;
    const int64_t total = (int64_t)L.M * K;
    const int32_t* slot = reinterpret_cast<const int32_t*>(blob + L.off_slot);
    const uint8_t* kind = blob + L.off_kind;
    const int n4 = L.nP + L.nF4;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        int m = (int)(i / K), idx = (int)(i % K);
        int kp = (idx % taps) * L.Cp + idx / taps;
        int p = slot[m], kd = kind[m];
        int v;
        if (kd == kFixed8)
            v = (int8_t)(blob + L.off_q8 + (size_t)(p - n4) * L.Kp)[kp];
        else
            v = decode4(blob + L.off_q4 + (size_t)p * (L.Kp / 2), kp, kd);
        values[i] = (int8_t)v;
        if (i < L.M) {
            if (perm) perm[i] = reinterpret_cast<const int32_t*>(blob + L.off_perm)[i];
            if (wstep) wstep[i] = reinterpret_cast<const float*>(blob + L.off_wstep)[i];
        }
    }
}

cudaError_t launch_unpack(const rmsmp_layer& L, const uint8_t* blob, int8_t* values,
                          int32_t* perm, float* wstep, cudaStream_t st)
{
    int64_t total = (int64_t)L.M * L.Cin * L.kh * L.kw;
    const int64_t cap = (int64_t)sm_count() * 16;
    int blocks = (int)((total + 255) / 256 < cap ? (total + 255) / 256 : cap);
    unpack_kernel<<<blocks, 256, 0, st>>>(blob, L, values, perm, wstep);
    return cudaGetLastError();
}

// ------------------------------------------------------------------ expand to int8 (workspace variant)
// One thread per 32 codes: a 128-bit load of packed 4-bit codes (or two of 8-bit codes) becomes two
// 128-bit stores of exact int8 values, rows in ORIGINAL order, reduction index as in the packed rows.

__global__ void __launch_bounds__(256) expand_kernel(const uint8_t* __restrict__ blob, rmsmp_layer L,
                                                     int8_t* __restrict__ wexp)
{
    const int chunks = L.Kp >> 5;
    const int64_t total = (int64_t)L.M * chunks;
    const int32_t* slot = reinterpret_cast<const int32_t*>(blob + L.off_slot);
    const uint8_t* kind = blob + L.off_kind;
    const int n4 = L.nP + L.nF4;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int m = (int)(i / chunks), c = (int)(i % chunks);
        const int p = slot[m], kd = kind[m];
        uint4 lo, hi;
        if (kd == kFixed8) {
            const uint4* src = reinterpret_cast<const uint4*>(blob + L.off_q8 + (size_t)(p - n4) * L.Kp + c * 32);
            lo = src[0]; hi = src[1];
        } else {
            const uint4 raw = *reinterpret_cast<const uint4*>(blob + L.off_q4 + (size_t)p * (L.Kp / 2) + c * 16);
            uint32_t w[8];
            if (kd == kPoT4) {
                expand_pot_chunk(raw, w);
            } else {
                // sign-extend the nibbles: (n ^ 8) - 8 per byte, done on 16 * value then shifted with sign
                expand_fixed4_chunk_x16(raw, w);
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const uint32_t x = w[q];
                    // arithmetic shift right by 4 of each byte: logical shift, then restore the sign bits
                    const uint32_t s = (x >> 4) & 0x0F0F0F0Fu;
                    const uint32_t neg = (x >> 7) & 0x01010101u;      // 1 where the byte is negative
                    w[q] = s | (neg * 0xF0u);
                }
            }
            lo = make_uint4(w[0], w[1], w[2], w[3]); hi = make_uint4(w[4], w[5], w[6], w[7]);
        }
        uint4* dst = reinterpret_cast<uint4*>(wexp + (size_t)m * L.Kp + c * 32);
        dst[0] = lo; dst[1] = hi;
    }
}

cudaError_t launch_expand(const rmsmp_layer& L, const uint8_t* blob, int8_t* wexp, cudaStream_t st)
{
    const int64_t total = (int64_t)L.M * (L.Kp >> 5);
    int64_t blocks = (total + 255) / 256;
    if (blocks > (int64_t)sm_count() * 8) blocks = (int64_t)sm_count() * 8;
    expand_kernel<<<(unsigned)blocks, 256, 0, st>>>(blob, L, wexp);
    return cudaGetLastError();
}

// ------------------------------------------------------------------ activation quantizer
// Pure streaming kernel.  The code is rint(clip(x / alpha) * Q) with ONE correctly rounded fp32
// division; that division costs more issue slots than the memory system leaves time for, so the
// vector path first forms the code from x * (1 / alpha) and keeps it only when the scaled value
// is not within 1e-4 of a rounding boundary (k + 0.5), where the two ways of computing x / alpha
// (relative difference < 2^-22) cannot round to different integers; the few values that are
// close to a boundary, and NaNs, take the division.  The results are those of act_code() in
// every case.

__device__ __forceinline__ uint32_t act_codes4(const float4& v, float alpha, int kind, const ActFast& f)
{
    bool redo = !f.ok;
    const uint32_t a = act_code_fast(v.x, f, redo), b = act_code_fast(v.y, f, redo),
                   c = act_code_fast(v.z, f, redo), d = act_code_fast(v.w, f, redo);
    if (redo)
        return (uint32_t)(act_code(v.x, alpha, kind) & 0xFF) | ((uint32_t)(act_code(v.y, alpha, kind) & 0xFF) << 8) |
               ((uint32_t)(act_code(v.z, alpha, kind) & 0xFF) << 16) | ((uint32_t)(act_code(v.w, alpha, kind) & 0xFF) << 24);
    return __byte_perm(__byte_perm(a, b, 0x0040), __byte_perm(c, d, 0x0040), 0x5410);
}

__global__ void __launch_bounds__(256) quantize_act_kernel(const float* __restrict__ x, size_t count,
                                                           float alpha, int kind,
                                                           int8_t* __restrict__ codes, int vec)
{
    const size_t tid = blockIdx.x * (size_t)blockDim.x + threadIdx.x;
    const size_t nthr = (size_t)gridDim.x * blockDim.x;
    if (vec) {
        // A warp takes 1024 consecutive values per step: eight 128-bit loads per lane, each
        // instruction covering 512 contiguous bytes, then eight 32-bit stores of 128 contiguous
        // bytes each.  The remaining 16-value groups follow one lane at a time.
        const size_t n16 = count / 16;
        const size_t n1024 = count / 1024;
        const int lane = threadIdx.x & 31;
        const size_t warp = tid >> 5, nwarp = nthr >> 5;
        const ActFast fast = act_fast_setup(alpha, kind);
        for (size_t i = warp; i < n1024; i += nwarp) {
            const float4* src = reinterpret_cast<const float4*>(x) + i * 256 + lane;
            float4 v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = __ldcs(src + j * 32);
            uint32_t* dst = reinterpret_cast<uint32_t*>(codes) + i * 256 + lane;
#pragma unroll
            for (int j = 0; j < 8; ++j) __stcs(dst + j * 32, act_codes4(v[j], alpha, kind, fast));
        }
        for (size_t i = n1024 * 64 + tid; i < n16; i += nthr) {
            const float4* src = reinterpret_cast<const float4*>(x) + i * 4;
            uint32_t w[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float4 v = src[j];
                w[j] = (uint32_t)(act_code(v.x, alpha, kind) & 0xFF) |
                       ((uint32_t)(act_code(v.y, alpha, kind) & 0xFF) << 8) |
                       ((uint32_t)(act_code(v.z, alpha, kind) & 0xFF) << 16) |
                       ((uint32_t)(act_code(v.w, alpha, kind) & 0xFF) << 24);
            }
            reinterpret_cast<uint4*>(codes)[i] = make_uint4(w[0], w[1], w[2], w[3]);
        }
        for (size_t i = n16 * 16 + tid; i < count; i += nthr) codes[i] = (int8_t)act_code(x[i], alpha, kind);
    } else {
        for (size_t i = tid; i < count; i += nthr) codes[i] = (int8_t)act_code(x[i], alpha, kind);
    }
}

cudaError_t launch_quantize_act(const float* x, size_t count, float alpha, int kind, int8_t* codes,
                                cudaStream_t st)
{
    int vec = ((reinterpret_cast<uintptr_t>(x) & 15) == 0 && (reinterpret_cast<uintptr_t>(codes) & 15) == 0);
    size_t steps = vec ? (count + 31) / 32 : count;      // the vector path handles 32 values per thread and step
    size_t blocks = (steps + 255) / 256;
    const size_t cap = (size_t)sm_count() * 32;
    if (blocks > cap) blocks = cap;
    if (blocks == 0) blocks = 1;
    quantize_act_kernel<<<(unsigned)blocks, 256, 0, st>>>(x, count, alpha, kind, codes, vec);
    return cudaGetLastError();
}

}  // namespace rmsmp
