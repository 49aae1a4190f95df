// Grouped weight-streaming kernel: many small-batch linear layers (up to 128 tokens each) in ONE
// launch on the tensor cores.
//
// With a handful of tokens a layer is bound by reading its packed weights once, and the only
// per-weight work is turning 4-bit codes into int8 operands.  One persistent CTA per SM walks its
// own list of work items.  An item is up to 128 (Fixed-8: 64) consecutive PACKED rows of ONE kind of one layer
// (the packed buffer groups the rows by kind, so such a tile is a dense block of the 4-bit or the
// 8-bit region), the whole reduction, all tokens.  Tiles of one kind keep the decode free of
// divergence and spread the expensive kind (PoT) evenly over the four SM sub-partitions; the
// price is an output scatter through the row permutation, which costs little with few tokens.
// Per item the reduction is cut into stages of 256 codes and at most 16 KB: ONE bulk copy of at most 128 rows x
// 128 bytes for a 4-bit tile; two of at most 64 rows x 128 bytes for an 8-bit tile, which is 64 rows high.  The
// expanded weights never touch shared memory: they go from registers to TENSOR MEMORY (tcgen05.st)
// and the MMA takes its A operand from there, so shared memory carries only the packed codes (once
// in, once out) and the activation tiles.  Warp roles:
//   warp 0       producer of the packed codes: one box per stage (128 / 64 / 32 rows high, whichever
//                covers the tile; 128-byte rows, 128-byte swizzle) into the packed-code ring.  A slot
//                is held from the start of its copy until the expanders have the bytes in registers,
//                i.e. for one trip to HBM: the ring's depth is what is in flight from HBM.
//   warp 1       producer of the activation codes: per k-block one swizzled box [n_pad tokens][128
//                codes] (rows beyond a layer's token count read zeros) into a ring of its own.
//   warps 2-3    idle (they keep the warp numbering of the roles below a multiple of four).
//   warps 4-7    MMA issuers.  tcgen05.mma, M = 128 rows, N = n_pad tokens, A from tensor memory, B
//                from shared memory, one instruction per 32 codes.  Fixed-4 and Fixed-8 tiles are
//                kind::i8 with int32 sums.  PoT-4 tiles are kind::f8f6f4: the code shifted left by two
//                is a 6-bit float (E3M2) of a quarter of its value, the activations are E4M3 bytes, the
//                sums are fp32 and exact (multiples of 1/4 below 2^22).  Activation bytes known to be
//                within 0..15 are read as they are (as an E4M3 number such a byte is the code times
//                2^-9, subnormals included); otherwise the E4M3 copy of a layer's codes is written
//                once per launch by a small kernel in front of this one (act_e4m3_kernel, into
//                scratch behind the table).  One thread gets an
//                MMA out only every ~150 cycles whatever its size (measured; two issuing threads
//                give twice the rate), so with few tokens the steps of a stage are dealt to up to
//                four issuers, each with an accumulator chain of its own (the chains are added up
//                in the epilogue).  Warp 4 allocates tensor memory.  Accumulator buffers take turns
//                between items so that an item's output overlaps the next items' stream.
//   warps 8-23   expanders, in two sets that take alternate stages (one set's waits fall into the
//                other's arithmetic).  A warp may touch the 32 tensor-memory lanes of its quarter
//                (warp % 4); thread <-> one row of the tile; a quarter's two warps of a set split
//                the stage's 32-code steps.  Consecutive lanes read consecutive rows of the
//                swizzled box (no bank conflicts).  16-byte raw chunk -> 32 int8 values in
//                registers -> tcgen05.st into the stage's columns.
//   warps 24-27  epilogue: tcgen05.ld, add the chains, undo the x16 of Fixed-4 rows (the 1/4 of PoT rows), scale by
//                wstep * act_step, and store each lane's value to its ORIGINAL row.
// Tensor memory: two or four accumulator buffers of nch * n_pad columns, then four to six A stages of 64 columns.
// The epilogue looks one item ahead for its rows' permutation entries and scales, which live in
// each layer's packed buffer; everything else an item needs is in the table.
// Every mbarrier wait is bounded; a wait that runs out sets the abort flag, all roles leave, tensor
// memory is freed and RMSMP_ERR_TIMEOUT is recorded in the current layer's status word.
#include <cuda.h>
#include <algorithm>
#include <cmath>
#include <cstring>
#include <queue>
#include <vector>
#include "common.cuh"
#include "decode.cuh"
#include "ptx.cuh"
#include "tmap.cuh"

namespace rmsmp {

namespace {

constexpr int kProdWarps = 4;                                         // warps 0-3: one kind of box each
constexpr int kMmaWarps = 4;                                          // warps 4-7: up to four MMA issuers
constexpr int kExpWarps = 16;                                         // warps 8-23
constexpr int kEpiWarps = 4;                                          // warps 24-27
constexpr int kFirstMma = kProdWarps, kFirstExp = kProdWarps + kMmaWarps, kFirstEpi = kFirstExp + kExpWarps;
constexpr int kStreamThreads = 32 * (kProdWarps + kMmaWarps + kExpWarps + kEpiWarps);      // 896
constexpr int kAStageCols = 64;                                       // 256 codes = 64 32-bit columns per lane
constexpr int kMaxTokens = 128;                                       // accumulator columns of one chain at most
constexpr int kRingMax = 12;
constexpr int kStreamMaxK = 16384;                                    // reduction length up to which the fp32 sums of PoT tiles are exact
constexpr int kLocalItems = 96;                                        // items of a CTA's list kept in shared memory
constexpr int kStreamSmem = 232448 - 1024 - kLocalItems * 16;
constexpr uint32_t kPlanMagic = 0x53545247u;                          // "STRG"

// One layer of the launch as the kernel sees it (device table, 128-byte aligned: it starts with
// the tensor maps).
struct alignas(128) StreamProblem {
    CUtensorMap q4[3], q8[3];       // packed 4-bit / 8-bit rows; boxes of 128, 64 and 32 rows x 128 bytes
    CUtensorMap act;                // activation codes [N][ld_act]; box n_pad tokens x 128 codes
    CUtensorMap act_fp;             // what the PoT tiles read: the E4M3 copy [N][Kp], or the codes themselves (act_nonneg)
    const int8_t* act_src;          // the codes, and where the copy goes (nullptr: no PoT rows)
    uint8_t* act_fp_dst;
    int64_t pix_pitch;
    int32_t Cin, Kp;
    const int32_t* perm;
    const float* wstep;
    float* out;
    int32_t* acc;
    uint32_t* status;
    int64_t ld_out;
    float act_step;
    int32_t M, N, nkb, out_mn;
    float fp_unit;                  // integer sum = fp32 sum of a PoT tile x this: 4 with the copy, 2^11 with raw bytes (code x 2^-9)
};
static_assert(sizeof(StreamProblem) % 128 == 0, "tensor maps stay 128-byte aligned in the array");

// One tile: `rows` (1..128) consecutive packed rows of one kind, starting at row `row0` of their storage
// region (4-bit or 8-bit) and at position `packed0` of the layer's permutation.
struct StreamItem { int32_t prob, kind_rows, row0, packed0; };      // kind_rows = kind << 28 | k-blocks of the layer << 8 | rows
__host__ __device__ inline int item_kind(int kr) { return (kr >> 28) & 3; }
__host__ __device__ inline int item_nkb(int kr) { return (kr >> 8) & 0xFFFFF; }
__host__ __device__ inline int item_rows(int kr) { return kr & 0xFF; }

struct StreamHeader {               // first 128 bytes of the table
    uint32_t magic;
    int32_t nprob, nitems, grid;
    int32_t n_pad, nS, nch, nB;               // tokens rounded up to 16, slots of the packed-code ring, accumulator chains (1, 2 or 4), slots of the activation ring
    uint32_t stage_bytes, b_bytes, idesc, smem_bytes;   // one slot of the packed-code ring / of the activation ring
    int32_t acc_cols, nAst;                   // tensor memory: columns of one accumulator buffer (nch * n_pad); A stages behind the two buffers
    uint32_t off_first, off_items, off_probs, bytes;
    uint32_t idesc_fp;                        // instruction descriptor of PoT tiles (E3M2 x E4M3 -> fp32)
    uint32_t off_act, n_fp;                   // scratch of the E4M3 activation copies; layers that have one
    uint32_t conv_grid_x;                     // blocks per layer of the kernel that writes them
    int32_t nAcc;                             // accumulator buffers in tensor memory (2 or 4): items in flight between issuers and epilogue
    uint32_t pad[9];
};
static_assert(sizeof(StreamHeader) == 128, "header is 128 bytes");

__host__ __device__ inline int box_index(int rows) { return rows > 64 ? 0 : (rows > 32 ? 1 : 2); }   // 128, 64 or 32 rows high

__device__ __forceinline__ void lds128(uint32_t addr, uint32_t& a, uint32_t& b, uint32_t& c, uint32_t& d)
{
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(a), "=r"(b), "=r"(c), "=r"(d) : "r"(addr) : "memory");
}

// A PoT-4 code (sign << 3 | e, value +-2^(e-1), e = 0: zero; Eq. 4) shifted left by two IS the 6-bit
// float with three exponent and two mantissa bits (bias 3, mantissa 00, exponent field 0 = zero) of a
// quarter of that value.  The tensor core takes such numbers in 8-bit containers (kind::f8f6f4, A format
// E3M2), multiplies exactly and adds in fp32, which is exact here: every product and every partial sum is
// a multiple of one unit (1/4, or 2^-11 with activation bytes read as they are) below 2^24 units (the host
// checks the reduction length).  So PoT rows need no table: two shifts and two masks spread the even and
// the odd codes of a word over two words, and two byte permutes put them back in order.
__device__ __forceinline__ void expand_pot_chunk_e3m2(const uint4& c, uint32_t out[8])
{
    const uint32_t x[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t ev = (x[i] << 2) & 0x3C3C3C3Cu, od = (x[i] >> 2) & 0x3C3C3C3Cu;
        out[2 * i] = prmt(ev, od, 0x5140u);
        out[2 * i + 1] = prmt(ev, od, 0x7362u);
    }
}

// Four int8 activation codes (each within -16..16) as four E4M3 bytes, exactly: byte + 128 is put under
// the fp16 exponent of 1024, 1152 is subtracted, and the pair is narrowed by the hardware conversion.
__device__ __forceinline__ uint32_t e4m3x4_of_s8x4(uint32_t w)
{
    const uint32_t u = w ^ 0x80808080u;
    uint32_t h01 = prmt(u, 0x64646464u, 0x5140u), h23 = prmt(u, 0x64646464u, 0x7362u), d;
    asm("{\n\t.reg .b16 lo, hi;\n\t"
        "sub.rn.f16x2 %1, %1, %3;\n\t"
        "sub.rn.f16x2 %2, %2, %3;\n\t"
        "cvt.rn.satfinite.e4m3x2.f16x2 lo, %1;\n\t"
        "cvt.rn.satfinite.e4m3x2.f16x2 hi, %2;\n\t"
        "mov.b32 %0, {lo, hi};\n\t}"
        : "=r"(d), "+r"(h01), "+r"(h23) : "r"(0x64806480u));
    return d;
}

// 32-byte piece `g` (0..3) of this thread's 128-byte raw row, expanded to 16 words of int8 values:
// a 4-bit row: its 32-code steps 2g and 2g + 1 (w[0..7], w[8..15]); an 8-bit row: its step g (w[0..7]; the
// rest is not used).  `row` = shared-memory address of the row, ph = its swizzle phase (row & 7).
template <int kind>
__device__ __forceinline__ void stream_expand(uint32_t row, uint32_t ph, int g, uint32_t (&w)[16])
{
    uint4 c0, c1;
    const uint32_t a0 = row + (((uint32_t)(2 * g) ^ ph) << 4);
    lds128(a0, c0.x, c0.y, c0.z, c0.w);
    lds128(a0 ^ 16u, c1.x, c1.y, c1.z, c1.w);
    if (kind == kFixed8) {
        w[0] = c0.x; w[1] = c0.y; w[2] = c0.z; w[3] = c0.w; w[4] = c1.x; w[5] = c1.y; w[6] = c1.z; w[7] = c1.w;
        return;
    }
    uint32_t lo[8], hi[8];
    if (kind == kPoT4) { expand_pot_chunk_e3m2(c0, lo); expand_pot_chunk_e3m2(c1, hi); }
    else { expand_fixed4_chunk_x16(c0, lo); expand_fixed4_chunk_x16(c1, hi); }
#pragma unroll
    for (int t = 0; t < 8; ++t) { w[t] = lo[t]; w[8 + t] = hi[t]; }
}

// 16 consecutive 32-bit columns of this thread's tensor-memory lane.
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&w)[16])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7]),
          "r"(w[8]), "r"(w[9]), "r"(w[10]), "r"(w[11]), "r"(w[12]), "r"(w[13]), "r"(w[14]), "r"(w[15])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// 16 accumulator columns of this thread's lane; valid after the wait.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr) : "memory");
}

// One MMA with the A operand in tensor memory (128 lanes x 8 columns = 128 rows x 32 codes) and the
// B operand in shared memory (descriptor given as 32-bit halves).
__device__ __forceinline__ void mma_i8_tmem_a(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi,
                                              uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], db, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
        : "memory");
}

// The same with E3M2 x E4M3 operands and fp32 accumulators.
__device__ __forceinline__ void mma_f8f6f4_tmem_a(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi,
                                                  uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], [%1], db, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
        : "memory");
}

// The tensor maps live in the table in global memory (written by a copy before the launch); fetching a
// tile's descriptor one tile ahead keeps its first copy from waiting for it.
__device__ __forceinline__ void tensormap_prefetch(const CUtensorMap* m)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(m) : "memory");
}
// E4M3 copies of the activation codes of every layer with PoT rows: [N][Kp], zeros beyond the layer's
// reduction length.  blockIdx.y = layer; layers whose bytes can be read as they are have no copy.
__global__ void __launch_bounds__(256) act_e4m3_kernel(const uint8_t* __restrict__ table)
{
    // Programmatic dependent launch on both sides: the streaming kernel behind this one may start at once, and
    // this kernel may have started before the launch in front of it (which may still read the copies) is over.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const StreamHeader* H = reinterpret_cast<const StreamHeader*>(table);
    const StreamProblem& P = reinterpret_cast<const StreamProblem*>(table + H->off_probs)[blockIdx.y];
    if (!P.act_fp_dst) return;
    const int upr = P.Kp >> 4;                            // 16-byte units per row
    const int units = P.N * upr;
    for (int u = blockIdx.x * 256 + threadIdx.x; u < units; u += gridDim.x * 256) {
        const int n = u / upr, k0 = (u - n * upr) << 4;
        const int8_t* src = P.act_src + (int64_t)n * P.pix_pitch + k0;
        uint4 v;
        if (k0 + 16 <= P.Cin) {
            v = *reinterpret_cast<const uint4*>(src);
        } else {
            uint32_t w[4] = {0u, 0u, 0u, 0u};
            for (int b = 0; b < 16 && k0 + b < P.Cin; ++b) w[b >> 2] |= (uint32_t)(uint8_t)src[b] << (8 * (b & 3));
            v = make_uint4(w[0], w[1], w[2], w[3]);
        }
        uint4 o;
        o.x = e4m3x4_of_s8x4(v.x); o.y = e4m3x4_of_s8x4(v.y);
        o.z = e4m3x4_of_s8x4(v.z); o.w = e4m3x4_of_s8x4(v.w);
        *reinterpret_cast<uint4*>(P.act_fp_dst + (int64_t)n * P.Kp + k0) = o;
    }
}

__global__ void __launch_bounds__(kStreamThreads, 1)
stream_kernel(const uint8_t* __restrict__ table)
{
    // The next launch on the stream may start while this one runs (programmatic dependent launch): its CTAs
    // take the SMs this launch's CTAs leave.  In turn this kernel may run beside the launch in front of it, so
    // what that launch may still read or write is touched only behind griddepcontrol.wait: the activation
    // copies (activation producer) and the outputs (epilogue).  Both roles exist in every CTA, so no CTA, and
    // hence no launch, ends before the launch in front of it has.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const StreamHeader* H = reinterpret_cast<const StreamHeader*>(table);
    const int32_t* cta_first = reinterpret_cast<const int32_t*>(table + H->off_first);
    const StreamItem* items = reinterpret_cast<const StreamItem*>(table + H->off_items);
    const StreamProblem* probs = reinterpret_cast<const StreamProblem*>(table + H->off_probs);
    const int n_pad = H->n_pad, nS = H->nS, nch = H->nch, nB = H->nB, nAst = H->nAst;
    const uint32_t stage_bytes = H->stage_bytes, b_bytes = H->b_bytes, idesc = H->idesc, idesc_fp = H->idesc_fp;
    const uint32_t acc_cols = (uint32_t)H->acc_cols, nAcc = (uint32_t)H->nAcc, a_base_col = nAcc * acc_cols;
    const uint32_t acc_shift = nAcc == 4u ? 2u : 1u;
    const uint32_t b_sub = (uint32_t)n_pad * 128u;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sB = smem_base;                        // activation ring
    const uint32_t sRing = sB + nB * b_bytes;             // packed-code ring
    const uint32_t sBar = sRing + nS * stage_bytes;
    const uint32_t bar_fullA = sBar, bar_emptyA = sBar + 8 * kRingMax;
    const uint32_t bar_full = sBar + 16 * kRingMax, bar_empty = sBar + 24 * kRingMax;
    const uint32_t bar_fullB = sBar + 32 * kRingMax;
    const uint32_t bar_tfull = sBar + 48 * kRingMax, bar_tempty = bar_tfull + 32;
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;
    __shared__ int4 s_items[kLocalItems];                 // the head of this CTA's list of items (prob, kind / k-blocks / rows, row0, packed0)

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int it0 = __ldg(cta_first + blockIdx.x), it1 = __ldg(cta_first + blockIdx.x + 1);
    for (int i = threadIdx.x; i < min(it1 - it0, kLocalItems); i += kStreamThreads) {
        s_items[i] = __ldg(reinterpret_cast<const int4*>(items + it0 + i));
    }

    int pf_it = it0, pf_st = 0;                           // thread 0: where its early copies stopped (item, stage)
    uint32_t pf_n = 0;                                    // ... and how many stages they were (at most one lap of the ring)
    if (threadIdx.x == 0) {
        for (int s = 0; s < kRingMax; ++s) {
            mbar_init(bar_fullA + 8 * s, kExpWarps / 2); // one arrival per expander warp of the set that has the stage
            mbar_init(bar_emptyA + 8 * s, 1);            // the tcgen05.commit of the stage's issuer: its A stage AND its activation slot are free
            mbar_init(bar_full + 8 * s, 1);              // the packed-code producer (+ transaction bytes)
            mbar_init(bar_empty + 8 * s, kExpWarps / 2); // the stage's expander warps, as soon as the codes are in their registers
            mbar_init(bar_fullB + 8 * s, 1);             // the activation producer (+ transaction bytes)
        }
        for (int b = 0; b < 4; ++b) {
            mbar_init(bar_tfull + 8 * b, nch);           // every issuer's tcgen05.commit
            mbar_init(bar_tempty + 8 * b, kEpiWarps);    // one arrival per epilogue warp
        }
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        // This thread is also the producer of the packed codes: the first lap of the ring needs no wait, so its copies
        // go out now, while the other warps are still setting up (tensor-memory allocation, the CTA-wide barrier).
        while (pf_it < it1 && pf_n < (uint32_t)nS) {
            const int4 a = __ldg(reinterpret_cast<const int4*>(items + pf_it));
            const int kind = item_kind(a.y), nkb = item_nkb(a.y), bi = box_index(item_rows(a.y));
            const bool two = kind == kFixed8;
            const int nst = (nkb + 1) >> 1;
            const StreamProblem* P = probs + a.x;
            const CUtensorMap* map = (kind == kFixed8) ? &P->q8[bi] : &P->q4[bi];
            const uint32_t tx = (uint32_t)(128 >> bi) * 128u;
            while (pf_st < nst && pf_n < (uint32_t)nS) {
                const uint32_t fbar = bar_full + 8 * pf_n;
                if (two) {
                    // an 8-bit tile of at most 64 rows: the stage's two k-blocks are two boxes, one per half of the slot
                    const int nb = min(2, nkb - 2 * pf_st);
                    mbar_arrive_expect_tx(fbar, (uint32_t)nb * tx);
                    for (int u = 0; u < nb; ++u)
                        tma_load_2d(sRing + pf_n * stage_bytes + (uint32_t)u * (stage_bytes >> 1), map, fbar, (2 * pf_st + u) * 128, a.z);
                } else {
                    mbar_arrive_expect_tx(fbar, tx);
                    tma_load_2d(sRing + pf_n * stage_bytes, map, fbar, pf_st * 128, a.z);
                }
                ++pf_st; ++pf_n;
            }
            if (pf_st == nst) { ++pf_it; pf_st = 0; }
        }
    }
    if (warp == kFirstMma) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&s_tmem_base)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = s_tmem_base;
    volatile int* abort_flag = &s_abort;

    uint32_t* last_status = nullptr;                      // status word of the layer this thread worked on last

    // An item's stages: two k-blocks (256 codes) each -- one box of a 4-bit tile, two boxes of an 8-bit tile.
    // The first kLocalItems items of the CTA's list were copied to shared memory above, with everything the
    // roles need to walk them, so that no role starts an item with a chain of dependent global loads.
    struct ItemView { const StreamProblem* P; int kind, rows, kbps, nst, nkb, row0, packed0; };
    auto view = [&](int it) -> ItemView {
        ItemView v;
        const int4 a = (it - it0 < kLocalItems) ? s_items[it - it0] : __ldg(reinterpret_cast<const int4*>(items + it));
        const int nkb = item_nkb(a.y);
        v.P = probs + a.x;
        v.kind = item_kind(a.y);
        v.rows = item_rows(a.y);
        v.row0 = a.z; v.packed0 = a.w;
        v.nkb = nkb;
        v.kbps = 2;                                      // k-blocks per stage: one box of a 4-bit tile, two boxes of an 8-bit tile
        v.nst = (nkb + 1) >> 1;
        return v;
    };

    if (warp == 0) {
        // ---------------------------------------------------------- producer of the packed codes (one lane)
        if (lane == 0) {
            uint32_t sr = pf_n == (uint32_t)nS ? 0u : pf_n, phR = pf_n == (uint32_t)nS ? 1u : 0u;
            bool ok = true;
            for (int it = pf_it; it < it1 && ok; ++it) {
                const ItemView v = view(it);
                last_status = v.P->status;
                const int bi = box_index(v.rows);
                const CUtensorMap* map = (v.kind == kFixed8) ? &v.P->q8[bi] : &v.P->q4[bi];
                if (it + 1 < it1) {
                    // fetch the next tile's descriptor now, so that its first copy does not wait for it
                    const ItemView nv = view(it + 1);
                    const int nb = box_index(nv.rows);
                    tensormap_prefetch((nv.kind == kFixed8) ? &nv.P->q8[nb] : &nv.P->q4[nb]);
                }
                const uint32_t tx = (uint32_t)(128 >> bi) * 128u;
                for (int st = (it == pf_it) ? pf_st : 0; st < v.nst; ++st) {
                    if (!mbar_wait_parked(bar_empty + 8 * sr, phR ^ 1, abort_flag)) { ok = false; break; }
                    const uint32_t fbar = bar_full + 8 * sr;
                    if (v.kind == kFixed8) {
                        const int nb = min(2, v.nkb - 2 * st);
                        mbar_arrive_expect_tx(fbar, (uint32_t)nb * tx);
                        for (int u = 0; u < nb; ++u)
                            tma_load_2d(sRing + sr * stage_bytes + (uint32_t)u * (stage_bytes >> 1), map, fbar, (2 * st + u) * 128, v.row0);
                    } else {
                        mbar_arrive_expect_tx(fbar, tx);
                        tma_load_2d(sRing + sr * stage_bytes, map, fbar, st * 128, v.row0);     // 128 bytes of every row per stage
                    }
                    if (++sr == (uint32_t)nS) { sr = 0; phR ^= 1; }
                }
            }
            if (!ok) {
                for (int i = 0; i < 200; ++i) __nanosleep(1000);   // let copies in flight land before the CTA's memory is released
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------- producer of the activation tiles (lanes 0 / 1: first / second k-block)
        uint32_t sb = 0, phB = 0;
        bool ok = true;
        // the E4M3 copies come from the kernel in front of this one
        asm volatile("griddepcontrol.wait;" ::: "memory");
        for (int it = it0; it < it1 && ok; ++it) {
            const ItemView v = view(it);
            last_status = v.P->status;
            const CUtensorMap* amap = (v.kind == kPoT4) ? &v.P->act_fp : &v.P->act;
            if (lane == 0 && it + 1 < it1) { const ItemView nv = view(it + 1); tensormap_prefetch(nv.kind == kPoT4 ? &nv.P->act_fp : &nv.P->act); }
            for (int st = 0; st < v.nst; ++st) {
                if (!mbar_wait_parked_warp(bar_emptyA + 8 * sb, phB ^ 1, abort_flag)) { ok = false; break; }    // activation slot s goes with A stage s
                const uint32_t fbar = bar_fullB + 8 * sb;
                const int kb0 = st * v.kbps;
                const int nsub = min(v.kbps, v.nkb - kb0);
                if (lane == 0) mbar_arrive_expect_tx(fbar, (uint32_t)nsub * b_sub);
                __syncwarp();
                if (lane < nsub) tma_load_2d(sB + sb * b_bytes + (uint32_t)lane * b_sub, amap, fbar, (kb0 + lane) * 128, 0);
                if (++sb == (uint32_t)nAst) { sb = 0; phB ^= 1; }
            }
        }
        if (!ok && lane == 0) {
            for (int i = 0; i < 200; ++i) __nanosleep(1000);
        }
    } else if (warp < kFirstMma) {
        // warps 2-3 have no role
    } else if (warp < kFirstExp) {
        // ---------------------------------------------------------- MMA issuers (lane 0 issues; the warp walks in step)
        // Every tcgen05 instruction holds its thread for ~150 cycles, the commit included, so a stage is one
        // issuer's: its four or eight MMAs and ONE commit, which frees the stage's A columns and activation slot.
        // The issuers take the CTA's stages in turn; stage st of an item adds to accumulator chain st % nch.
        const int me = warp - kFirstMma;
        if (me < nch) {
            const bool issuer = (lane == 0);
            uint32_t sa = (uint32_t)me, phA = 0, n = 0, t = 0;        // t: stages of the items before this one
            const uint64_t desc_b0 = smem_desc_kmajor(sB, 128);
            const uint32_t b_lo0 = (uint32_t)desc_b0, desc_hi = (uint32_t)(desc_b0 >> 32);
            bool ok = true;
            for (int it = it0; it < it1 && ok && !*abort_flag; ++it, ++n) {
                const ItemView v = view(it);
                last_status = v.P->status;
                const uint32_t ab = n & (nAcc - 1u), lap = n >> acc_shift;      // nAcc is 2 or 4
                bool have_acc = false;                    // this issuer has made sure the item's accumulator buffer is free
                // its own stages only: those whose index over the whole list is me modulo nch (1, 2 or 4); the A stage
                // advances by nch with them (nch <= nAst)
                for (int st = (int)(((uint32_t)me - t) & (uint32_t)(nch - 1)); st < v.nst; st += nch) {
                    {
                        if (!have_acc) {
                            if (!mbar_wait_parked(bar_tempty + 8 * ab, (lap & 1) ^ 1, abort_flag)) { ok = false; break; }
                            have_acc = true;
                        }
                        if (!mbar_wait_parked(bar_fullB + 8 * sa, phA, abort_flag) || !mbar_wait_parked(bar_fullA + 8 * sa, phA, abort_flag)) { ok = false; break; }
                        tc_fence_after();
                        if (issuer) {
                            const uint32_t chain = (uint32_t)st & (uint32_t)(nch - 1);
                            const uint32_t d_tmem = tmem_base + ab * acc_cols + chain * (uint32_t)n_pad;
                            const uint32_t a_t = tmem_base + a_base_col + sa * kAStageCols, b_lo = b_lo0 + sa * (b_bytes >> 4);
                            // a 32-code step is 8 columns of A and 32 bytes (two 16-byte units) of a B row; the first
                            // instruction into a chain in this item overwrites it
                            const int nsteps = 4 * min(v.kbps, v.nkb - st * v.kbps);
                            if (v.kind == kPoT4) {
                                for (int j = 0; j < nsteps; ++j) {
                                    const uint32_t b_j = b_lo + (uint32_t)(j >> 2) * (b_sub >> 4) + 2u * (uint32_t)(j & 3);
                                    mma_f8f6f4_tmem_a(d_tmem, a_t + 8 * j, b_j, desc_hi, idesc_fp, (st < nch && j == 0) ? 0u : 1u);
                                }
                            } else {
                                for (int j = 0; j < nsteps; ++j) {
                                    const uint32_t b_j = b_lo + (uint32_t)(j >> 2) * (b_sub >> 4) + 2u * (uint32_t)(j & 3);
                                    mma_i8_tmem_a(d_tmem, a_t + 8 * j, b_j, desc_hi, idesc, (st < nch && j == 0) ? 0u : 1u);
                                }
                            }
                            mma_commit(bar_emptyA + 8 * sa);
                        }
                    }
                    sa += (uint32_t)nch;
                    if (sa >= (uint32_t)nAst) { sa -= (uint32_t)nAst; phA ^= 1; }
                }
                t += (uint32_t)v.nst;
                if (!ok) break;
                // Every issuer reports once per item, whether or not a stage of it was its own.  An issuer without
                // stages in short items can be items ahead of the others: before it reports on this buffer again
                // it makes sure that the buffer's previous item has everybody's report (one arrival per phase).
                if (lap >= 1 && !mbar_wait_parked(bar_tfull + 8 * ab, (lap - 1) & 1, abort_flag)) break;
                if (issuer) mma_commit(bar_tfull + 8 * ab);
            }
        }
    } else if (warp < kFirstEpi) {
        // ---------------------------------------------------------- expanders
        // The sixteen warps form two sets that take alternate stages, so that one set's waits (for the
        // copy engine, for a free tensor-memory stage, for its stores) fall into the other set's arithmetic;
        // inside a set a quarter's two warps split the stage's 128-byte rows in halves.
        const int quarter = warp & 3;                    // tensor-memory lanes 32 * quarter .. + 31
        const int set = ((warp - kFirstExp) >> 2) & 1;   // which stages: those with (stage index & 1) == set
        const int half = (warp - kFirstExp) >> 3;        // which half of a raw row: its 32-byte pieces 2 * half, 2 * half + 1
        const int slot = quarter * 32 + lane;            // the thread's row of every tile
        const uint32_t row_off = (uint32_t)slot * 128u, ph = (uint32_t)(slot & 7);
        const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16) + a_base_col;
        uint32_t t = 0;                                  // stages of the items before the current one
        // ring positions of the set's next stage: its stages are every other one of the CTA's list, so both rings
        // advance by two with them (nS >= 2, nAst even)
        uint32_t sr = (uint32_t)set, phR = 0, sa = (uint32_t)set, phA = 0;
        auto advance = [&]() {
            sr += 2u; if (sr >= (uint32_t)nS) { sr -= (uint32_t)nS; phR ^= 1; }
            sa += 2u; if (sa >= (uint32_t)nAst) { sa -= (uint32_t)nAst; phA ^= 1; }
        };
        bool ok = true;
        for (int it = it0; it < it1 && ok; ++it) {
            const ItemView v = view(it);
            last_status = v.P->status;
            const bool have_row = slot < v.rows;         // lanes beyond the tile's rows hand zeros to the MMA
            const bool eight = v.kind == kFixed8;
            for (int st = (int)(((uint32_t)set - t) & 1u); st < v.nst; st += 2) {
                {
                    if (!mbar_wait_parked_warp(bar_full + 8 * sr, phR, abort_flag)) { ok = false; break; }
                    const uint32_t row = sRing + sr * stage_bytes + row_off;
                    uint32_t w[16], w2[16];
                    if (eight) {
                        // An 8-bit tile has at most 64 rows (tensor-memory lanes 0..63: quarters 0 and 1); its stage is
                        // two boxes, one per k-block.  A 32-byte piece g of a row is its 32-code step g: 8 columns.
                        // w[0..7] / w[8..15]: this thread's two pieces of the first / of the second box.
                        const int nb = min(2, v.nkb - 2 * st);
                        if (have_row) {
                            stream_expand<kFixed8>(row, ph, 2 * half, w);
                            stream_expand<kFixed8>(row, ph, 2 * half + 1, w2);
#pragma unroll
                            for (int q = 0; q < 8; ++q) w[8 + q] = w2[q];
                            if (nb == 2) {
                                uint32_t x[16];
                                stream_expand<kFixed8>(row + (stage_bytes >> 1), ph, 2 * half, w2);
                                stream_expand<kFixed8>(row + (stage_bytes >> 1), ph, 2 * half + 1, x);
#pragma unroll
                                for (int q = 0; q < 8; ++q) w2[8 + q] = x[q];
                            }
                        } else {
#pragma unroll
                            for (int q = 0; q < 16; ++q) { w[q] = 0u; w2[q] = 0u; }
                        }
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar_empty + 8 * sr);
                        if (!mbar_wait_parked_warp(bar_emptyA + 8 * sa, phA ^ 1, abort_flag)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t col8 = t_lane + sa * kAStageCols;
                        tmem_st16(col8 + 16 * half, w);                    // first k-block: columns 0..31
                        if (nb == 2) tmem_st16(col8 + 32 + 16 * half, w2);  // second k-block: columns 32..63
                        tmem_st_wait();
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar_fullA + 8 * sa);
                        advance();
                        continue;
                    }
                    if (have_row && v.kind == kPoT4) {
                        stream_expand<kPoT4>(row, ph, 2 * half, w);
                        stream_expand<kPoT4>(row, ph, 2 * half + 1, w2);
                    } else if (have_row) {
                        stream_expand<kFixed4>(row, ph, 2 * half, w);
                        stream_expand<kFixed4>(row, ph, 2 * half + 1, w2);
                    } else {
#pragma unroll
                        for (int q = 0; q < 16; ++q) { w[q] = 0u; w2[q] = 0u; }
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_empty + 8 * sr);       // the raw bytes are in registers: the slot can be refilled
                    if (!mbar_wait_parked_warp(bar_emptyA + 8 * sa, phA ^ 1, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t col = t_lane + sa * kAStageCols;
                    // a 4-bit row's 32-byte piece g is its steps 2g, 2g + 1: 16 columns
                    tmem_st16(col + 32 * half, w);
                    tmem_st16(col + 32 * half + 16, w2);
                    tmem_st_wait();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_fullA + 8 * sa);
                }
                advance();
            }
            t += (uint32_t)v.nst;
        }
    } else {
        // ---------------------------------------------------------- epilogue
        const int quarter = warp & 3;                    // tensor-memory lanes this warp may read
        const int slot = quarter * 32 + lane;
        uint32_t n = 0;
        bool alive = true;
        // this lane's row of an item: original index, scale and Fixed-4 shift, fetched ahead of the accumulator
        auto row_info = [&](int it, float& scale, int& shift, int& m) {
            scale = 0.f; shift = 0; m = -1;
            if (it >= it1) return;
            const ItemView v = view(it);
            if (slot < v.rows) {
                m = __ldg(v.P->perm + v.packed0 + slot);
                scale = __fmul_rn(__ldg(v.P->wstep + m), v.P->act_step);
                shift = (v.kind == kFixed4) ? 4 : 0;     // expanders store Fixed-4 codes as 16 * value
            }
        };
        float scale, scale_n; int shift, shift_n, m, m_n;
        row_info(it0, scale, shift, m);
        asm volatile("griddepcontrol.wait;" ::: "memory");      // the launch in front of this one may still be writing the same outputs
        for (int it = it0; it < it1 && alive; ++it, ++n) {
            const ItemView vi = view(it);
            const StreamProblem* P = vi.P;
            last_status = P->status;
            row_info(it + 1, scale_n, shift_n, m_n);
            const uint32_t ab = n & (nAcc - 1u);
            if (!mbar_wait_parked_warp(bar_tfull + 8 * ab, (n >> acc_shift) & 1, abort_flag)) { alive = false; break; }
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + ab * acc_cols;
            const int N = P->N;
            const int nchains = min(nch, vi.nst);                // chains this item's stages went to
            float* const out = P->out;
            int32_t* const acc = P->acc;
            const int64_t ld = P->ld_out;
            const bool out_mn = P->out_mn != 0;
            // one value of this lane's row: undo the x16 of Fixed-4 rows, scale, store (and the raw sum if asked for)
            // this lane's row: where its value of token nn goes
            const int64_t o_row = out_mn ? (int64_t)m * ld : (int64_t)m, o_tok = out_mn ? 1 : ld;
            auto put = [&](int nn, uint32_t raw) {
                const int a = (int)raw >> shift;
                const int64_t o = o_row + (int64_t)nn * o_tok;
                out[o] = __fmul_rn(__int2float_rn(a), scale);
                if (acc) acc[o] = a;
            };
            auto release_tmem = [&]() {
                // every accumulator of this item is in registers: hand the buffer back
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_tempty + 8 * ab);
            };
            // 16 tokens at a time; with few tokens the 32-code steps went to nch accumulator chains in turn: add them
            const int n16 = (N + 15) >> 4;
            const bool fp = vi.kind == kPoT4;            // fp32 sums: add the chains (exactly), then the integer number of units
            const float fp_unit = P->fp_unit;
            for (int ch = 0; ch < n16; ++ch) {
                uint32_t v[16];
                tmem_ld16(taddr + ch * 16, v);
                for (int c = 1; c < nchains; ++c) {
                    uint32_t u[16];
                    tmem_ld16(taddr + c * n_pad + ch * 16, u);
                    if (fp) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) v[j] = __float_as_uint(__fadd_rn(__uint_as_float(v[j]), __uint_as_float(u[j])));
                    } else {
#pragma unroll
                        for (int j = 0; j < 16; ++j) v[j] += u[j];
                    }
                }
                if (fp) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] = (uint32_t)__float2int_rn(__fmul_rn(__uint_as_float(v[j]), fp_unit));
                }
                if (ch == n16 - 1) release_tmem();
                if (m < 0) continue;
                const int jmax = min(16, N - ch * 16);
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    if (j < jmax) put(ch * 16 + j, v[j]);
            }
            scale = scale_n; shift = shift_n; m = m_n;
        }
    }

    // ---------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == kFirstMma) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
    }
    if (s_abort && last_status && lane == 0) atomicMax(last_status, (uint32_t)RMSMP_ERR_TIMEOUT);
}

// ------------------------------------------------------------------ host side

inline size_t up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Layout {
    int grid, nitems;
    size_t off_first, off_items, off_probs, off_act, bytes;      // bytes: the table proper; the E4M3 copies follow at off_act
};

Layout table_layout(int count, int nitems, int grid)
{
    Layout L;
    L.grid = grid; L.nitems = nitems;
    size_t off = sizeof(StreamHeader);
    L.off_first = off; off = up(off + sizeof(int32_t) * (size_t)(grid + 1), 16);
    L.off_items = off; off = up(off + sizeof(StreamItem) * (size_t)nitems, 128);
    L.off_probs = off; off += sizeof(StreamProblem) * (size_t)count;
    L.bytes = up(off, 256);
    L.off_act = L.bytes;
    return L;
}

}  // namespace

// Height of a Fixed-8 tile: 64 rows, two k-blocks (two boxes of 64 rows x 128 bytes) per stage, so that a stage of
// any tile is 16 KB and 256 codes deep.  Measured against 128-row tiles with one k-block per stage on the paper's
// mix: 46 against 47.4 us at 8 tokens (half as many stages for the few Fixed-8 rows of a layer; the idle
// tensor-memory quarters cost nothing).  A layer of Fixed-8 rows only, which no ratio of the paper is, pays for it
// (72 against 61 us).
static int f8_tile_rows(int, int, int) { return 64; }

// Tiles of a layer: the rows of each 4-bit kind in blocks of 128 packed rows, the 8-bit rows in blocks of 64 or 128.
int64_t stream_items_of(int nP, int nF4, int n8)
{
    const int t8 = f8_tile_rows(nP, nF4, n8);
    return (nP + 127) / 128 + (nF4 + 127) / 128 + (n8 + t8 - 1) / t8;
}

// Scratch bytes the table of `count` layers with `nitems` tiles needs on a device with `sms` SMs.
size_t stream_table_bytes(int count, int64_t nitems, int sms, int64_t act_bytes)
{
    return table_layout(count, (int)nitems, sms).bytes + (size_t)act_bytes;
}

// Bytes of the E4M3 activation copy of one layer (0 without PoT rows).
int64_t stream_act_bytes(int nP, int act_nonneg, int64_t N, int Kp)
{
    return (nP > 0 && !act_nonneg) ? (int64_t)up((size_t)(N * Kp), 256) : 0;
}

// Can this problem be part of a grouped tensor-core launch?
bool stream_supported(const Problem& p)
{
    if (p.kh != 1 || p.kw != 1 || p.N < 1 || p.N > kMaxTokens) return false;
    if (p.pix_pitch % 16 != 0 || (reinterpret_cast<uintptr_t>(p.act) & 15) != 0) return false;
    // PoT tiles are summed in fp32 in units of 1/4: exact while 64 * 16 * K <= 2^24
    if (p.nP > 0 && p.Kp > kStreamMaxK) return false;
    if (p.Kp / 128 >= (1 << 20)) return false;                  // the k-block count travels in 20 bits of an item's word
    return tensor_map_encoder() != nullptr;
}

// Builds the table on the host (`h_table`, stream_table_bytes(...) bytes) and the launch geometry.
// Returns false if a tensor map cannot be encoded or the shared-memory budget does not fit.
bool stream_build_table(const Problem* probs, int count, int sms, uint8_t* h_table, size_t table_bytes,
                        uint8_t* d_table, int* grid_out, uint32_t* smem_out, uint32_t* conv_grid_out)
{
    EncodeTiledFn enc = tensor_map_encoder();
    if (!enc) return false;
    int64_t nitems = 0;
    int64_t maxN = 1;
    for (int i = 0; i < count; ++i) {
        nitems += stream_items_of(probs[i].nP, probs[i].nF4, probs[i].n8);
        maxN = std::max<int64_t>(maxN, probs[i].N);
    }
    if (nitems >= (1ll << 30)) return false;
    const int grid = (int)std::min<int64_t>(sms, nitems);
    const Layout L = table_layout(count, (int)nitems, grid);
    int64_t act_bytes = 0;
    for (int i = 0; i < count; ++i) act_bytes += stream_act_bytes(probs[i].nP, probs[i].act_nonneg, probs[i].N, probs[i].Kp);
    if (L.bytes + (size_t)act_bytes > table_bytes) return false;
    memset(h_table, 0, L.bytes);
    StreamHeader* H = reinterpret_cast<StreamHeader*>(h_table);
    H->magic = kPlanMagic; H->nprob = count; H->nitems = (int32_t)nitems; H->grid = grid;
    H->n_pad = std::max(16, (int)((maxN + 15) / 16 * 16));
    // consecutive MMAs of one thread are ~150 cycles apart; with few tokens the accumulator buffer has room
    // for several chains, one per issuing thread (summed in the epilogue)
    H->nch = H->n_pad <= 32 ? 4 : (H->n_pad <= 64 ? 2 : 1);
    H->acc_cols = H->nch * H->n_pad;                              // <= 128
    // a short item's output (tensor-memory loads, scattered stores) takes about as long as its stream: with four
    // accumulator buffers the issuers do not wait for it
    H->nAcc = H->acc_cols <= 64 ? 4 : 2;
    H->nAst = std::min(6, (512 - H->nAcc * H->acc_cols) / kAStageCols) & ~1;      // even: the two expander sets alternate
    // An issuer waits on the barriers of its own stages only and tells their phases apart by parity, so it must never
    // skip two phases of a barrier: not more issuers than A stages, and an even number of A stages (each expander set
    // and each issuer then keeps to its own ones).
    if (H->nAst < H->nch || H->nAst < 2) return false;
    H->b_bytes = (uint32_t)(2 * H->n_pad * 128);
    H->stage_bytes = 128u * 128u;                                 // one box: at most 128 rows x 128 bytes
    // Shared memory: a packed-code slot is held from the moment its copy is started until the expanders have the
    // bytes in registers, i.e. for one trip to HBM, so the number of such slots is what is in flight from HBM; an
    // activation slot is held until its MMAs have finished and goes with the A stage of the same index.  The
    // packed codes get everything else.
    const int64_t avail = kStreamSmem - 1024 - 64 * kRingMax;
    H->nB = H->nAst;                                               // activation slot s goes with A stage s (one commit frees both)
    H->nS = (int)std::min<int64_t>(kRingMax, (avail - (int64_t)H->nB * H->b_bytes) / H->stage_bytes);
    if (H->nS < 2) return false;
    H->smem_bytes = (uint32_t)(H->nB * H->b_bytes + H->nS * H->stage_bytes + 1024 + 64 * kRingMax);
    // kind::i8: int32 accumulate, signed 8-bit A and B, both K-major, N/8 at bit 17, M/16 at bit 24
    H->idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(H->n_pad >> 3) << 17) | ((uint32_t)(kBlockRows >> 4) << 24);
    // kind::f8f6f4: fp32 accumulate (1 at bit 4), A = E3M2 (4 at bit 7), B = E4M3 (0 at bit 10)
    H->idesc_fp = (1u << 4) | (4u << 7) | (0u << 10) | ((uint32_t)(H->n_pad >> 3) << 17) | ((uint32_t)(kBlockRows >> 4) << 24);
    H->off_first = (uint32_t)L.off_first; H->off_items = (uint32_t)L.off_items; H->off_probs = (uint32_t)L.off_probs;
    H->bytes = (uint32_t)L.bytes;
    H->off_act = (uint32_t)L.off_act;

    // problems and their tensor maps
    StreamProblem* sp = reinterpret_cast<StreamProblem*>(h_table + L.off_probs);
    size_t act_off = 0;
    int64_t max_units = 0;
    for (int i = 0; i < count; ++i) {
        const Problem& p = probs[i];
        StreamProblem& q = sp[i];
        auto make_w = [&](CUtensorMap* m, const uint8_t* base, int rows, int pitch, int box_rows) -> bool {
            if (rows <= 0) return true;
            const cuuint64_t gd[2] = {(cuuint64_t)pitch, (cuuint64_t)rows};
            const cuuint64_t gs[1] = {(cuuint64_t)pitch};
            const cuuint32_t bx[2] = {128u, (cuuint32_t)box_rows};
            const cuuint32_t es[2] = {1, 1};
            return enc(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(base), gd, gs, bx, es,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
        };
        for (int b = 0; b < 3; ++b)
            if (!make_w(&q.q4[b], p.q4, p.nP + p.nF4, p.Kp / 2, 128 >> b) || !make_w(&q.q8[b], p.q8, p.n8, p.Kp, 128 >> b))
                return false;
        {
            const cuuint64_t gd[2] = {(cuuint64_t)p.Cin, (cuuint64_t)p.N};
            const cuuint64_t gs[1] = {(cuuint64_t)p.pix_pitch};
            const cuuint32_t bx[2] = {128u, (cuuint32_t)H->n_pad};
            const cuuint32_t es[2] = {1, 1};
            if (enc(&q.act, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t*>(p.act), gd, gs, bx, es,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
                return false;
        }
        q.fp_unit = p.act_nonneg ? 2048.0f : 4.0f;
        if (p.nP > 0 && p.act_nonneg) {
            q.act_fp = q.act;
        } else if (p.nP > 0) {
            q.act_src = p.act;
            q.act_fp_dst = d_table + L.off_act + act_off;
            q.pix_pitch = p.pix_pitch; q.Cin = p.Cin; q.Kp = p.Kp;
            act_off += (size_t)stream_act_bytes(p.nP, p.act_nonneg, p.N, p.Kp);
            H->n_fp += 1;
            max_units = std::max<int64_t>(max_units, p.N * (int64_t)(p.Kp / 16));
            const cuuint64_t gd[2] = {(cuuint64_t)p.Kp, (cuuint64_t)p.N};
            const cuuint64_t gs[1] = {(cuuint64_t)p.Kp};
            const cuuint32_t bx[2] = {128u, (cuuint32_t)H->n_pad};
            const cuuint32_t es[2] = {1, 1};
            if (enc(&q.act_fp, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, q.act_fp_dst, gd, gs, bx, es,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
                return false;
        }
        q.perm = p.perm; q.wstep = p.wstep;
        q.out = p.out; q.acc = p.acc; q.status = p.status; q.ld_out = p.ld_out;
        q.act_step = p.act_step; q.M = p.M; q.N = (int32_t)p.N;
        q.nkb = p.Kp / 128; q.out_mn = p.out_mn;
    }

    H->conv_grid_x = (uint32_t)std::max<int64_t>(1, std::min<int64_t>(64, (max_units + 255) / 256));

    // work items: every tile of every layer, handed to the CTAs longest first onto the least loaded one; an
    // item's cost is its stages, weighted by kind and box height, plus a constant for start-up and output
    struct Cand { int64_t cost; StreamItem item; };
    std::vector<Cand> cand;
    cand.reserve((size_t)nitems);
    for (int i = 0; i < count; ++i) {
        const Problem& p = probs[i];
        const int nkb = p.Kp / 128;
        const int n_of[3] = {p.nP, p.nF4, p.n8};
        const int region_row0[3] = {0, p.nP, 0};                   // first row of the kind inside its storage region
        const int perm0[3] = {0, p.nP, p.nP + p.nF4};              // ... and inside the permutation
        const int tile_rows[3] = {128, 128, f8_tile_rows(p.nP, p.nF4, p.n8)};
        for (int k = 0; k < 3; ++k)
            for (int r = 0; r < n_of[k]; r += tile_rows[k]) {
                const int rows = std::min(tile_rows[k], n_of[k] - r);
                const int nst = (nkb + 1) / 2;
                // measured: a stage of a full PoT / Fixed-4 / Fixed-8 tile takes about 1.11 : 1 : 1.1, half of it whatever
                // the height of its box; an item's start-up and output about 3/4 of a full stage
                static const int kind_weight[3] = {111, 100, 110};
                const int64_t cost = (int64_t)nst * kind_weight[k] * (64 + (64 >> box_index(rows))) + 9600;
                cand.push_back({cost, {i, (k << 28) | (nkb << 8) | rows, region_row0[k] + r, perm0[k] + r}});
            }
    }
    std::stable_sort(cand.begin(), cand.end(), [](const Cand& a, const Cand& b) { return a.cost > b.cost; });
    typedef std::pair<int64_t, int> Load;                  // (assigned cost, CTA)
    std::priority_queue<Load, std::vector<Load>, std::greater<Load>> heap;
    for (int c = 0; c < grid; ++c) heap.push({0, c});
    std::vector<std::vector<StreamItem>> lists((size_t)grid);
    for (const Cand& cd : cand) {
        Load l = heap.top();
        heap.pop();
        lists[(size_t)l.second].push_back(cd.item);
        heap.push({l.first + cd.cost, l.second});
    }
    int32_t* first = reinterpret_cast<int32_t*>(h_table + L.off_first);
    StreamItem* out_items = reinterpret_cast<StreamItem*>(h_table + L.off_items);
    int pos = 0;
    for (int c = 0; c < grid; ++c) {
        first[c] = pos;
        // within a CTA keep the layers in the order they were given
        std::stable_sort(lists[(size_t)c].begin(), lists[(size_t)c].end(),
                         [](const StreamItem& a, const StreamItem& b) { return a.prob != b.prob ? a.prob < b.prob : a.packed0 < b.packed0; });
        for (const StreamItem& it : lists[(size_t)c]) out_items[pos++] = it;
    }
    first[grid] = pos;
    *grid_out = grid;
    *smem_out = H->smem_bytes;
    if (H->n_fp == 0) H->conv_grid_x = 0;
    *conv_grid_out = H->conv_grid_x;
    return true;
}

// Both kernels are launched as programmatic dependents of whatever is in front of them on the stream.
// conv_grid_x > 0: layers with PoT rows are part of the launch; their activation copies are written first.
cudaError_t launch_stream(const uint8_t* d_table, int grid, uint32_t smem_bytes, int count, uint32_t conv_grid_x, cudaStream_t st)
{
    static bool attr_set[kMaxDevices] = {};
    if (!ensure_smem_attr(reinterpret_cast<const void*>(stream_kernel), kStreamSmem, attr_set)) return cudaErrorUnknown;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.stream = st; cfg.attrs = at; cfg.numAttrs = 1;
    if (conv_grid_x != 0) {
        cfg.gridDim = dim3(conv_grid_x, (unsigned)count); cfg.blockDim = dim3(256); cfg.dynamicSmemBytes = 0;
        cudaError_t e = cudaLaunchKernelEx(&cfg, act_e4m3_kernel, d_table);
        if (e != cudaSuccess) return e;
    }
    cfg.gridDim = dim3((unsigned)grid); cfg.blockDim = dim3(kStreamThreads); cfg.dynamicSmemBytes = smem_bytes;
    return cudaLaunchKernelEx(&cfg, stream_kernel, d_table);
}

}  // namespace rmsmp
