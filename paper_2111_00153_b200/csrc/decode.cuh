// Register-level expansion of one 16-byte packed chunk (32 four-bit codes) into 32 int8
// values held in eight 32-bit words, in reduction order.  Used by the CUDA-core kernels and
// by the expander warps of the tensor-core kernel.
#pragma once
#include <stdint.h>

namespace rmsmp {

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

// PoT-4: nibble i of a word is code i (sign<<3 | e).  The magnitude 0,1,2,...,64 comes from an
// 8-entry byte table indexed by e through a byte permute; the negative table is selected where
// the sign bit is set (sign masks are built with the permute's sign-replicate mode).
__device__ __forceinline__ void expand_pot_word(uint32_t x, uint32_t& v0123, uint32_t& v4567)
{
    const uint32_t kPosLo = 0x04020100u, kPosHi = 0x40201008u;   // 0,1,2,4 | 8,16,32,64
    const uint32_t kNegLo = 0xFCFEFF00u, kNegHi = 0xC0E0F0F8u;   // 0,-1,-2,-4 | -8,-16,-32,-64
    const uint32_t e = x & 0x77777777u;
    const uint32_t y = x << 4;
    const uint32_t eh = e >> 16;
    const uint32_t pa = prmt(kPosLo, kPosHi, e), pb = prmt(kPosLo, kPosHi, eh);
    const uint32_t na = prmt(kNegLo, kNegHi, e), nb = prmt(kNegLo, kNegHi, eh);
    const uint32_t sa = prmt(y, x, 0xD9C8u), sb = prmt(y, x, 0xFBEAu);
    v0123 = (pa & ~sa) | (na & sa);
    v4567 = (pb & ~sb) | (nb & sb);
}

// Exact values of a PoT chunk: out[0..7] hold codes 0..31 in order.
__device__ __forceinline__ void expand_pot_chunk(const uint4& c, uint32_t out[8])
{
    expand_pot_word(c.x, out[0], out[1]);
    expand_pot_word(c.y, out[2], out[3]);
    expand_pot_word(c.z, out[4], out[5]);
    expand_pot_word(c.w, out[6], out[7]);
}

// Fixed-4: byte b of the chunk holds code b in its high and code 16+b in its low nibble.
// Moving a nibble to the high half of a byte gives 16 * value as an int8, exactly; the caller
// divides the finished sum by 16 (an arithmetic shift: the sum of multiples of 16 is one).
__device__ __forceinline__ void expand_fixed4_chunk_x16(const uint4& c, uint32_t out[8])
{
    out[0] = c.x & 0xF0F0F0F0u; out[1] = c.y & 0xF0F0F0F0u;
    out[2] = c.z & 0xF0F0F0F0u; out[3] = c.w & 0xF0F0F0F0u;
    out[4] = (c.x << 4) & 0xF0F0F0F0u; out[5] = (c.y << 4) & 0xF0F0F0F0u;
    out[6] = (c.z << 4) & 0xF0F0F0F0u; out[7] = (c.w << 4) & 0xF0F0F0F0u;
}

}  // namespace rmsmp
