// The 4-bit activation quantizer's per-value arithmetic, shared by the streaming quantizer kernel
// and the re-quantizing epilogue of the contraction kernel.
#pragma once
#include "common.cuh"

namespace rmsmp {

// The definition: rint(clip(x / alpha) * Q) with ONE correctly rounded fp32 division.
__device__ __forceinline__ int act_code(float x, float alpha, int kind)
{
    float t = __fdiv_rn(x, alpha);
    if (kind == RMSMP_ACT_U4) {
        t = fminf(fmaxf(t, 0.0f), 1.0f);
        return __float2int_rn(__fmul_rn(t, 15.0f));
    }
    t = fminf(fmaxf(t, -1.0f), 1.0f);
    return __float2int_rn(__fmul_rn(t, 7.0f));
}

struct ActFast {
    float r, lo, q;        // 1 / alpha, lower clip, levels per unit
    bool ok;               // alpha is far from the ends of the fp32 range, so r is accurate
};

__device__ __forceinline__ ActFast act_fast_setup(float alpha, int kind)
{
    ActFast f;
    f.r = __frcp_rn(alpha);
    f.lo = (kind == RMSMP_ACT_U4) ? 0.0f : -1.0f;
    f.q = (kind == RMSMP_ACT_U4) ? 15.0f : 7.0f;
    f.ok = (alpha > 1e-30f) && (alpha < 1e30f);
    return f;
}

// Code of x in the low byte of the result; sets `redo` when the division has to decide: the scaled
// value here and the one the definition forms differ by a few roundings of relative size 2^-24
// (< 1e-5 absolute at Q = 15), so they round to the same integer whenever this one is further
// than 1e-4 from a rounding boundary k + 0.5.
__device__ __forceinline__ uint32_t act_code_fast(float x, const ActFast& f, bool& redo)
{
    const float kMagic = 12582912.0f;                       // 1.5 * 2^23: adding it rounds to an integer, half to even
    float t = __fmul_rn(x, f.r);
    t = fminf(fmaxf(t, f.lo), 1.0f);
    const float u = __fmul_rn(t, f.q);
    const float s = __fadd_rn(u, kMagic);
    const float c = __fsub_rn(s, kMagic);
    redo = redo || !(fabsf(__fsub_rn(u, c)) <= 0.4999f);      // also true for NaN
    return __float_as_uint(s);                               // low byte = the integer, two's complement
}


// One value by the fast path, by the definition where the fast path does not decide.
__device__ __forceinline__ uint32_t act_code_exact(float x, float alpha, int kind, const ActFast& f)
{
    bool redo = !f.ok;
    uint32_t c = act_code_fast(x, f, redo);
    if (redo) c = (uint32_t)act_code(x, alpha, kind);
    return c;
}

}  // namespace rmsmp
