// Grouped weight-streaming kernel: many small-batch linear layers (up to 128 tokens each) in ONE
// launch on the tensor cores.
//
// With a handful of tokens a layer is bound by reading its packed weights once, and the only
// per-weight work is turning 4-bit codes into int8 operands.  One persistent CTA per SM walks its
// own list of work items; an item is one block of 128 ORIGINAL rows of one layer (the three runs
// of the packed buffer that hold those rows), the whole reduction, all tokens.  Per item the
// reduction is cut into stages of two k-blocks (256 codes).  The expanded weights never touch
// shared memory: they go from registers to TENSOR MEMORY (tcgen05.st) and the MMA takes its A
// operand from there, so shared memory carries only the packed codes (once in, once out) and the
// activation tiles.  With the A operand staged in shared memory the kernel was bound by that
// memory's port (every weight byte crossed it four more times, expanded).  Warp roles:
//   warps 0-3    producers, one kind of box each: the item's PoT run, its Fixed-4 run, its Fixed-8
//                run (one box per k-block) and the activation codes (one box [n_pad tokens][128
//                codes] per k-block; rows beyond a layer's token count read zeros).  A run is ONE
//                box of 128-byte rows with the 128-byte swizzle, as high as the longest such run
//                of any block of the layer.  Starting a bulk copy holds the issuing thread for a
//                hundred cycles and more, whatever the copy's size, so the boxes are few and
//                large and are started by different warps.  Packed codes and activations of a
//                stage share one ring slot and one "full" barrier.
//   warps 4-7    MMA issuers.  tcgen05.mma kind::i8, M = 128 rows, N = n_pad tokens, A from tensor
//                memory, B from shared memory, eight instructions per stage.  One thread gets an
//                MMA out only every ~150 cycles whatever its size (measured; two issuing threads
//                give twice the rate), so with few tokens the eight 32-code steps of a stage are
//                dealt to up to four issuers, each with an accumulator chain of its own (the
//                chains are added up in the epilogue).  Warp 4 allocates tensor memory.
//                Accumulator buffers alternate between items so that an item's output overlaps
//                the next item's stream.
//   warps 8-23   expanders.  A warp may touch the 32 tensor-memory lanes of its quarter (warp % 4);
//                the four warps of a quarter split a stage's eight 32-code steps.  Thread <-> one
//                row: lane i of the accumulator is the i-th row of the item in packed order (PoT
//                rows, Fixed-4 rows, Fixed-8 rows), so a warp's lanes are rows of one kind (no
//                divergence except where two runs meet) and read consecutive rows of a swizzled
//                box (no bank conflicts).  16-byte raw chunk -> 32 int8 values in registers ->
//                tcgen05.st into the stage's 64 columns.
//   warps 24-27  epilogue: tcgen05.ld, add the chains, undo the x16 of Fixed-4 rows, scale by
//                wstep * act_step, and store each lane's value to its ORIGINAL row (the 128 rows
//                of an item are 128 adjacent outputs of a token, so the stores stay inside one
//                512-byte window).
// Tensor memory: two accumulator buffers of nch * n_pad columns, then four to six A stages of 64 columns.
// Every role looks one item ahead for the small per-item metadata (block table entry, row
// permutation, row scales), which lives in each layer's packed buffer.
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
constexpr int kStreamSmem = 232448 - 1024;
constexpr uint32_t kPlanMagic = 0x53545247u;                          // "STRG"

// One layer of the launch as the kernel sees it (device table, 128-byte aligned: it starts with
// the tensor maps).
struct alignas(128) StreamProblem {
    CUtensorMap q4p, q4f, q8, act;  // packed 4-bit rows (box height of the PoT / Fixed-4 runs), packed 8-bit rows, activation codes [N][ld_act]
    const int32_t* perm;
    const float* wstep;
    const uint8_t* kind;
    const int32_t* blocks;
    float* out;
    int32_t* acc;
    uint32_t* status;
    int64_t ld_out;
    float act_step;
    int32_t M, N, nP, nF4, nkb, out_mn;
    int32_t hP, hF, hE;             // box heights: rows of the longest PoT / Fixed-4 / Fixed-8 run of any block, rounded up to 8
    int32_t pad0[3];
};
static_assert(sizeof(StreamProblem) % 128 == 0, "tensor maps stay 128-byte aligned in the array");

struct StreamItem { int32_t prob, blk; };

struct StreamHeader {               // first 128 bytes of the table
    uint32_t magic;
    int32_t nprob, nitems, grid;
    int32_t n_pad, nS, nch, nB;               // tokens rounded up to 16, slots of the packed-code ring, accumulator chains (1, 2 or 4), slots of the activation ring
    uint32_t stage_bytes, b_bytes, idesc, smem_bytes;   // one slot of the packed-code ring / of the activation ring
    int32_t acc_cols, nAst;                   // tensor memory: columns of one accumulator buffer (nch * n_pad); A stages behind the two buffers
    uint32_t off_first, off_items, off_probs, bytes;
    uint32_t pad[14];
};
static_assert(sizeof(StreamHeader) == 128, "header is 128 bytes");

struct BlockRuns { int p0, nP, f0, nF, e0, nE; };
__device__ __forceinline__ BlockRuns load_runs(const StreamProblem* P, int blk)
{
    const int4 b0 = __ldg(reinterpret_cast<const int4*>(P->blocks + 8 * blk));
    const int2 b1 = __ldg(reinterpret_cast<const int2*>(P->blocks + 8 * blk + 4));
    BlockRuns b;
    b.p0 = b0.x; b.nP = b0.y; b.f0 = b0.z; b.nF = b0.w; b.e0 = b1.x; b.nE = b1.y;
    return b;
}

// What an expander thread knows about its row of an item: bits 0-15 byte offset, inside the packed-
// code part of a ring slot, of the 128-byte box row that holds the thread's two 32-code steps (for
// an 8-bit row: of the box row of the k-block those steps lie in), bits 16-18 the row's swizzle phase
// (row & 7 inside its box), bits 30-31 kind (3: no such row).  g = which pair of steps (0..3) the
// thread's warp takes.
__device__ __forceinline__ uint32_t stream_meta(const StreamProblem* P, int blk, int slot, int g)
{
    if (P == nullptr) return 3u << 30;
    const BlockRuns b = load_runs(P, blk);
    int kind, raw, r;
    if (slot < b.nP) {
        kind = kPoT4; r = slot; raw = r * 128;
    } else if (slot < b.nP + b.nF) {
        kind = kFixed4; r = slot - b.nP; raw = (P->hP + r) * 128;
    } else if (slot < b.nP + b.nF + b.nE) {
        kind = kFixed8; r = slot - b.nP - b.nF;
        raw = (P->hP + P->hF + (g >> 1) * P->hE + r) * 128;       // 8-bit rows: one box per k-block
    } else {
        return 3u << 30;
    }
    return (uint32_t)raw | ((uint32_t)(r & 7) << 16) | ((uint32_t)kind << 30);
}

// Original row (inside the layer) of accumulator lane `slot` of an item, or -1.
__device__ __forceinline__ int stream_row(const StreamProblem* P, int blk, int slot, int& kind)
{
    const BlockRuns b = load_runs(P, blk);
    int packed;
    if (slot < b.nP) { kind = kPoT4; packed = b.p0 + slot; }
    else if (slot < b.nP + b.nF) { kind = kFixed4; packed = P->nP + b.f0 + (slot - b.nP); }
    else if (slot < b.nP + b.nF + b.nE) { kind = kFixed8; packed = P->nP + P->nF4 + b.e0 + (slot - b.nP - b.nF); }
    else { kind = 3; return -1; }
    return __ldg(P->perm + packed);
}

__device__ __forceinline__ void lds128(uint32_t addr, uint32_t& a, uint32_t& b, uint32_t& c, uint32_t& d)
{
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(a), "=r"(b), "=r"(c), "=r"(d) : "r"(addr) : "memory");
}

// The thread's two 32-code steps of this stage, expanded: w[0..7] = step 2g, w[8..15] = step 2g + 1.
__device__ __forceinline__ void stream_expand(uint32_t meta, uint32_t raw_stage, int g, uint32_t (&w)[16])
{
    const uint32_t kind = meta >> 30;
    const uint32_t row = raw_stage + (meta & 0xFFFFu);
    const uint32_t ph = (meta >> 16) & 7u;
    if (kind == kFixed8) {
        // steps 2g, 2g + 1 are the four 16-byte chunks 4 (g & 1) .. + 3 of the row's k-block
        const uint32_t j0 = 4u * (uint32_t)(g & 1);
#pragma unroll
        for (int t = 0; t < 4; ++t) lds128(row + (((j0 + t) ^ ph) << 4), w[4 * t], w[4 * t + 1], w[4 * t + 2], w[4 * t + 3]);
        return;
    }
    if (kind == 3u) {
#pragma unroll
        for (int t = 0; t < 16; ++t) w[t] = 0u;
        return;
    }
    uint4 c0, c1;
    const uint32_t a0 = row + (((uint32_t)(2 * g) ^ ph) << 4);
    lds128(a0, c0.x, c0.y, c0.z, c0.w);
    lds128(a0 ^ 16u, c1.x, c1.y, c1.z, c1.w);
    uint32_t lo[8], hi[8];
    if (kind == kPoT4) { expand_pot_chunk(c0, lo); expand_pot_chunk(c1, hi); }
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

__device__ __forceinline__ void tensormap_acquire(const CUtensorMap* m)
{
    asm volatile("fence.proxy.tensormap::generic.acquire.gpu [%0], 128;" ::"l"(m) : "memory");
}

__global__ void __launch_bounds__(kStreamThreads, 1)
stream_kernel(const uint8_t* __restrict__ table)
{
    const StreamHeader* H = reinterpret_cast<const StreamHeader*>(table);
    const int32_t* cta_first = reinterpret_cast<const int32_t*>(table + H->off_first);
    const StreamItem* items = reinterpret_cast<const StreamItem*>(table + H->off_items);
    const StreamProblem* probs = reinterpret_cast<const StreamProblem*>(table + H->off_probs);
    const int n_pad = H->n_pad, nS = H->nS, nch = H->nch, nB = H->nB, nAst = H->nAst;
    const uint32_t stage_bytes = H->stage_bytes, b_bytes = H->b_bytes, idesc = H->idesc;
    const uint32_t acc_cols = (uint32_t)H->acc_cols, a_base_col = 2u * acc_cols;
    const uint32_t b_sub = (uint32_t)n_pad * 128u;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sB = smem_base;                        // activation ring
    const uint32_t sRing = sB + nB * b_bytes;             // packed-code ring
    const uint32_t sBar = sRing + nS * stage_bytes;
    const uint32_t bar_fullA = sBar, bar_emptyA = sBar + 8 * kRingMax;
    const uint32_t bar_full = sBar + 16 * kRingMax, bar_empty = sBar + 24 * kRingMax;
    const uint32_t bar_fullB = sBar + 32 * kRingMax, bar_emptyB = sBar + 40 * kRingMax;
    const uint32_t bar_tfull = sBar + 48 * kRingMax, bar_tempty = bar_tfull + 16;
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kRingMax; ++s) {
            mbar_init(bar_fullA + 8 * s, kExpWarps / 2); // one arrival per expander warp of the set that has the stage
            mbar_init(bar_emptyA + 8 * s, nch);          // every issuer's tcgen05.commit
            mbar_init(bar_full + 8 * s, kProdWarps - 1); // the three producer warps of the packed codes (+ their transaction bytes)
            mbar_init(bar_empty + 8 * s, kExpWarps / 2); // the stage's expander warps, as soon as the codes are in their registers
            mbar_init(bar_fullB + 8 * s, 1);             // the activation producer (+ transaction bytes)
            mbar_init(bar_emptyB + 8 * s, nch);          // every issuer's tcgen05.commit
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_tfull + 8 * b, nch);           // every issuer's tcgen05.commit
            mbar_init(bar_tempty + 8 * b, kEpiWarps);    // one arrival per epilogue warp
        }
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
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

    const int it0 = __ldg(cta_first + blockIdx.x), it1 = __ldg(cta_first + blockIdx.x + 1);
    uint32_t* last_status = nullptr;                      // status word of the layer this thread worked on last

    if (warp < kProdWarps) {
        // ---------------------------------------------------------- producers
        // warp 0: the PoT run; warp 1: the Fixed-4 run; warp 2: the Fixed-8 run, lanes 0 / 1 the stage's first /
        // second k-block; warp 3: the activation tiles, lanes 0 / 1 likewise
        uint32_t sr = 0, phR = 0;
        bool ok = true;
        int prev_prob = -1;
        struct Box { const CUtensorMap* map; int row; uint32_t dst, tx; };      // tx: bytes of this WARP's boxes per stage
        auto box_of = [&](int it) -> Box {
            Box bx = {nullptr, 0, 0u, 0u};
            if (it >= it1) return bx;
            const StreamItem item = items[it];
            const StreamProblem* P = probs + item.prob;
            const BlockRuns br = load_runs(P, item.blk);
            if (warp == 0) {
                bx.tx = (uint32_t)P->hP * 128u;
                if (lane == 0 && P->hP) { bx.map = &P->q4p; bx.row = br.p0; bx.dst = 0u; }
            } else if (warp == 1) {
                bx.tx = (uint32_t)P->hF * 128u;
                if (lane == 0 && P->hF) { bx.map = &P->q4f; bx.row = P->nP + br.f0; bx.dst = (uint32_t)P->hP * 128u; }
            } else if (warp == 2) {
                bx.tx = 2u * (uint32_t)P->hE * 128u;
                if (lane < 2 && P->hE) { bx.map = &P->q8; bx.row = br.e0; bx.dst = (uint32_t)(P->hP + P->hF + lane * P->hE) * 128u; }
            } else {
                bx.tx = b_sub;                            // per k-block
                if (lane < 2) { bx.map = &P->act; bx.row = 0; bx.dst = (uint32_t)lane * b_sub; }
            }
            return bx;
        };
        Box cur = box_of(it0);
        for (int it = it0; it < it1 && ok; ++it) {
            const StreamItem item = items[it];
            const StreamProblem* P = probs + item.prob;
            last_status = P->status;
            if (item.prob != prev_prob) {
                // the maps were written to the table by an earlier kernel: order this thread's use of them after that
                if (cur.map) tensormap_acquire(cur.map);
                prev_prob = item.prob;
            }
            const Box nxt = box_of(it + 1);               // in flight while this item streams
            const int nkb = P->nkb, npairs = (nkb + 1) >> 1;
            // warps 0-2 fill the packed-code ring, warp 3 the activation ring (its own depth and barriers)
            const uint32_t ring_n = (warp == 3) ? (uint32_t)nB : (uint32_t)nS;
            const uint32_t bar_e = (warp == 3) ? bar_emptyB : bar_empty, bar_f = (warp == 3) ? bar_fullB : bar_full;
            const uint32_t ring0 = (warp == 3) ? sB : sRing, ring_b = (warp == 3) ? b_bytes : stage_bytes;
            for (int kp = 0; kp < npairs; ++kp) {
                if (!mbar_wait_parked_warp(bar_e + 8 * sr, phR ^ 1, abort_flag)) { ok = false; break; }
                const uint32_t fbar = bar_f + 8 * sr;
                const bool two = 2 * kp + 1 < nkb;
                if (lane == 0) mbar_arrive_expect_tx(fbar, (warp == 3 && two) ? 2u * cur.tx : cur.tx);
                __syncwarp();
                // byte offset into the source row: 4-bit runs 128 bytes per stage; 8-bit runs and activations 128 per k-block
                const int x = (warp < 2) ? kp * 128 : (2 * kp + lane) * 128;
                if (cur.map && !(warp == 3 && lane == 1 && !two))
                    tma_load_2d(ring0 + sr * ring_b + cur.dst, cur.map, fbar, x, cur.row);
                if (++sr == ring_n) { sr = 0; phR ^= 1; }
            }
            cur = nxt;
        }
        if (!ok && lane == 0) {
            for (int i = 0; i < 200; ++i) __nanosleep(1000);   // let copies in flight land before the CTA's memory is released
        }
    } else if (warp < kFirstExp) {
        // ---------------------------------------------------------- MMA issuers (lane 0 issues; the warp walks in step)
        const int me = warp - kFirstMma;                  // issuer me takes the 32-code steps me, me + nch, ... into chain me
        if (me < nch) {
            const bool issuer = (lane == 0);
            uint32_t sa = 0, phA = 0, sb = 0, phB = 0, n = 0;
            const uint64_t desc_b0 = smem_desc_kmajor(sB, 128);
            const uint32_t b_lo0 = (uint32_t)desc_b0, desc_hi = (uint32_t)(desc_b0 >> 32);
            bool ok = true;
            for (int it = it0; it < it1 && ok && !*abort_flag; ++it, ++n) {
                const StreamItem item = items[it];
                const StreamProblem* P = probs + item.prob;
                last_status = P->status;
                const int nkb = P->nkb, npairs = (nkb + 1) >> 1;
                const uint32_t ab = n & 1;
                if (!mbar_wait_parked(bar_tempty + 8 * ab, ((n >> 1) & 1) ^ 1, abort_flag)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + ab * acc_cols + (uint32_t)(me * n_pad);
                for (int kp = 0; kp < npairs; ++kp) {
                    if (!mbar_wait_parked(bar_fullB + 8 * sb, phB, abort_flag) || !mbar_wait_parked(bar_fullA + 8 * sa, phA, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_t = tmem_base + a_base_col + sa * kAStageCols, b_lo = b_lo0 + sb * (b_bytes >> 4);
                    if (issuer) {
                        // a 32-code step is 8 columns of A and 32 bytes (two 16-byte units) of a B row; this
                        // issuer's first instruction of the item overwrites its chain
                        const int nsteps = (2 * kp + 1 < nkb) ? 8 : 4;
                        for (int j = me; j < nsteps; j += nch) {
                            const uint32_t b_j = b_lo + (uint32_t)(j >> 2) * (b_sub >> 4) + 2u * (uint32_t)(j & 3);
                            mma_i8_tmem_a(d_tmem, a_t + 8 * j, b_j, desc_hi, idesc, (kp == 0 && j == me) ? 0u : 1u);
                        }
                        mma_commit(bar_emptyA + 8 * sa);
                        mma_commit(bar_emptyB + 8 * sb);
                    }
                    if (++sa == (uint32_t)nAst) { sa = 0; phA ^= 1; }
                    if (++sb == (uint32_t)nB) { sb = 0; phB ^= 1; }
                }
                if (!ok) break;
                if (issuer) mma_commit(bar_tfull + 8 * ab);
            }
        }
    } else if (warp < kFirstEpi) {
        // ---------------------------------------------------------- expanders
        // The sixteen warps form two sets that take alternate stages, so that one set's waits (for the
        // copy engine, for a free tensor-memory stage, for its stores) fall into the other set's arithmetic;
        // inside a set a quarter's two warps split the stage's two k-blocks.
        const int quarter = warp & 3;                    // tensor-memory lanes 32 * quarter .. + 31
        const int set = ((warp - kFirstExp) >> 2) & 1;   // which stages: those with (stage index & 1) == set
        const int half = (warp - kFirstExp) >> 3;        // which k-block of a stage: its 32-code steps 4 * half .. + 3
        const int slot = quarter * 32 + lane;            // the thread's row of every item, in packed order
        const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16) + a_base_col + 32 * half;
        uint32_t t = 0;                                  // stages this CTA has been through
        uint32_t sr = 0, phR = 0, sa = 0, phA = 0;       // ring positions of stage t (advanced for every stage, taken or not)
        auto meta_of = [&](int it) -> uint32_t {
            if (it >= it1) return 3u << 30;
            const StreamItem item = items[it];
            return stream_meta(probs + item.prob, item.blk, slot, 2 * half);
        };
        uint32_t cur = meta_of(it0);
        bool ok = true;
        for (int it = it0; it < it1 && ok; ++it) {
            const StreamItem item = items[it];
            const StreamProblem* P = probs + item.prob;
            last_status = P->status;
            const int npairs = (P->nkb + 1) >> 1;
            const uint32_t nxt = meta_of(it + 1);         // in flight during this item
            for (int kp = 0; kp < npairs; ++kp, ++t) {
                if ((int)(t & 1u) == set) {
                    if (!mbar_wait_parked_warp(bar_full + 8 * sr, phR, abort_flag)) { ok = false; break; }
                    const uint32_t raw = sRing + sr * stage_bytes;
                    uint32_t w[16];
                    stream_expand(cur, raw, 2 * half, w);
                    if (!mbar_wait_parked_warp(bar_emptyA + 8 * sa, phA ^ 1, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    tmem_st16(t_lane + sa * kAStageCols, w);
                    stream_expand(cur, raw, 2 * half + 1, w);
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_empty + 8 * sr);       // the raw bytes are in registers: the slot can be refilled
                    tmem_st16(t_lane + sa * kAStageCols + 16, w);
                    tmem_st_wait();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_fullA + 8 * sa);
                }
                if (++sr == (uint32_t)nS) { sr = 0; phR ^= 1; }
                if (++sa == (uint32_t)nAst) { sa = 0; phA ^= 1; }
            }
            cur = nxt;
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
            const StreamItem item = items[it];
            const StreamProblem* P = probs + item.prob;
            int kind;
            m = stream_row(P, item.blk, slot, kind);
            if (m >= 0) {
                scale = __fmul_rn(__ldg(P->wstep + m), P->act_step);
                shift = (kind == kFixed4) ? 4 : 0;       // expanders store Fixed-4 codes as 16 * value
            }
        };
        float scale, scale_n; int shift, shift_n, m, m_n;
        row_info(it0, scale, shift, m);
        for (int it = it0; it < it1 && alive; ++it, ++n) {
            const StreamItem item = items[it];
            const StreamProblem* P = probs + item.prob;
            last_status = P->status;
            row_info(it + 1, scale_n, shift_n, m_n);
            const uint32_t ab = n & 1;
            if (!mbar_wait_parked_warp(bar_tfull + 8 * ab, (n >> 1) & 1, abort_flag)) { alive = false; break; }
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + ab * acc_cols;
            const int N = P->N;
            float* const out = P->out;
            int32_t* const acc = P->acc;
            const int64_t ld = P->ld_out;
            const bool out_mn = P->out_mn != 0;
            // one value of this lane's row: undo the x16 of Fixed-4 rows, scale, store (and the raw sum if asked for)
            auto put = [&](int nn, uint32_t raw) {
                const int a = (int)raw >> shift;
                const int64_t o = out_mn ? (int64_t)m * ld + nn : (int64_t)nn * ld + m;
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
            for (int ch = 0; ch < n16; ++ch) {
                uint32_t v[16];
                tmem_ld16(taddr + ch * 16, v);
                for (int c = 1; c < nch; ++c) {
                    uint32_t u[16];
                    tmem_ld16(taddr + c * n_pad + ch * 16, u);
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] += u[j];
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
    size_t off_first, off_items, off_probs, bytes;
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
    return L;
}

}  // namespace

// Scratch bytes the table of `count` layers with `nitems` row blocks needs on a device with `sms` SMs.
size_t stream_table_bytes(int count, int64_t nitems, int sms)
{
    return table_layout(count, (int)nitems, sms).bytes;
}

// Can this problem be part of a grouped tensor-core launch?
bool stream_supported(const Problem& p)
{
    if (p.kh != 1 || p.kw != 1 || p.N < 1 || p.N > kMaxTokens) return false;
    if (p.pix_pitch % 16 != 0 || (reinterpret_cast<uintptr_t>(p.act) & 15) != 0) return false;
    if (p.max_blk[0] + p.max_blk[1] + p.max_blk[2] <= 0) return false;      // descriptor from an older rmsmp_layer_init
    return tensor_map_encoder() != nullptr;
}

// Builds the table on the host (`h_table`, stream_table_bytes(...) bytes, device address `d_table` for nothing
// but alignment checks) and the launch geometry.  Returns false if a tensor map cannot be encoded or the
// shared-memory budget does not fit.
bool stream_build_table(const Problem* probs, int count, int sms, uint8_t* h_table, size_t table_bytes,
                        int* grid_out, uint32_t* smem_out)
{
    EncodeTiledFn enc = tensor_map_encoder();
    if (!enc) return false;
    int64_t nitems = 0;
    int64_t maxN = 1;
    int raw_rows = 0;                                    // 128-byte box rows of packed codes per stage, largest layer
    auto up8 = [](int n) { return (n + 7) / 8 * 8; };
    for (int i = 0; i < count; ++i) {
        nitems += probs[i].nblocks;
        maxN = std::max<int64_t>(maxN, probs[i].N);
        raw_rows = std::max(raw_rows, up8(probs[i].max_blk[0]) + up8(probs[i].max_blk[1]) + 2 * up8(probs[i].max_blk[2]));
    }
    if (nitems >= (1ll << 30)) return false;
    const int grid = (int)std::min<int64_t>(sms, nitems);
    const Layout L = table_layout(count, (int)nitems, grid);
    if (L.bytes > table_bytes) return false;
    memset(h_table, 0, L.bytes);
    StreamHeader* H = reinterpret_cast<StreamHeader*>(h_table);
    H->magic = kPlanMagic; H->nprob = count; H->nitems = (int32_t)nitems; H->grid = grid;
    H->n_pad = std::max(16, (int)((maxN + 15) / 16 * 16));
    // consecutive MMAs into one accumulator wait for each other; with few tokens the accumulator buffer has room
    // for several chains that the 32-code steps take in turn (summed in the epilogue)
    H->nch = H->n_pad <= 32 ? 4 : (H->n_pad <= 64 ? 2 : 1);
    H->acc_cols = H->nch * H->n_pad;                              // <= 128
    H->nAst = std::min(6, (512 - 2 * H->acc_cols) / kAStageCols) & ~1;      // even: the two expander sets alternate
    H->b_bytes = (uint32_t)(2 * H->n_pad * 128);
    H->stage_bytes = (uint32_t)raw_rows * 128u;                   // multiples of 1024: every box starts on a swizzle atom
    // Shared memory: a packed-code slot is held from the moment its copy is started until the expanders have the
    // bytes in registers, i.e. for one trip to HBM, so the number of such slots is what is in flight from HBM; an
    // activation slot is held until its MMAs have finished.  Activations get up to six slots (a quarter of the
    // memory at most), the packed codes everything else.
    const int64_t avail = kStreamSmem - 1024 - 64 * kRingMax;
    H->nB = (int)std::min<int64_t>(6, std::max<int64_t>(2, avail / 4 / H->b_bytes));
    H->nS = (int)std::min<int64_t>(kRingMax, (avail - (int64_t)H->nB * H->b_bytes) / H->stage_bytes);
    if (H->nS < 2) return false;
    H->smem_bytes = (uint32_t)(H->nB * H->b_bytes + H->nS * H->stage_bytes + 1024 + 64 * kRingMax);
    // kind::i8: int32 accumulate, signed 8-bit A and B, both K-major, N/8 at bit 17, M/16 at bit 24
    H->idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(H->n_pad >> 3) << 17) | ((uint32_t)(kBlockRows >> 4) << 24);
    H->off_first = (uint32_t)L.off_first; H->off_items = (uint32_t)L.off_items; H->off_probs = (uint32_t)L.off_probs;
    H->bytes = (uint32_t)L.bytes;

    // problems and their tensor maps
    StreamProblem* sp = reinterpret_cast<StreamProblem*>(h_table + L.off_probs);
    for (int i = 0; i < count; ++i) {
        const Problem& p = probs[i];
        StreamProblem& q = sp[i];
        q.hP = up8(p.max_blk[0]); q.hF = up8(p.max_blk[1]); q.hE = up8(p.max_blk[2]);
        auto make_w = [&](CUtensorMap* m, const uint8_t* base, int rows, int pitch, int box_rows) -> bool {
            if (rows <= 0 || box_rows <= 0) return true;
            const cuuint64_t gd[2] = {(cuuint64_t)pitch, (cuuint64_t)rows};
            const cuuint64_t gs[1] = {(cuuint64_t)pitch};
            const cuuint32_t bx[2] = {128u, (cuuint32_t)box_rows};
            const cuuint32_t es[2] = {1, 1};
            return enc(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(base), gd, gs, bx, es,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
        };
        if (!make_w(&q.q4p, p.q4, p.nP + p.nF4, p.Kp / 2, q.hP) || !make_w(&q.q4f, p.q4, p.nP + p.nF4, p.Kp / 2, q.hF) ||
            !make_w(&q.q8, p.q8, p.n8, p.Kp, q.hE))
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
        q.perm = p.perm; q.wstep = p.wstep; q.kind = p.kind; q.blocks = p.blocks;
        q.out = p.out; q.acc = p.acc; q.status = p.status; q.ld_out = p.ld_out;
        q.act_step = p.act_step; q.M = p.M; q.N = (int32_t)p.N; q.nP = p.nP; q.nF4 = p.nF4;
        q.nkb = p.Kp / 128; q.out_mn = p.out_mn;
    }

    // work items: every row block of every layer, handed to the CTAs longest first onto the least loaded
    // one; an item's cost is its number of stages plus a constant for start-up and output
    struct Cand { int64_t cost; int prob, blk; };
    std::vector<Cand> cand;
    cand.reserve((size_t)nitems);
    for (int i = 0; i < count; ++i) {
        const int npairs = (probs[i].Kp / 128 + 1) / 2;
        for (int b = 0; b < probs[i].nblocks; ++b) cand.push_back({(int64_t)npairs + 2, i, b});
    }
    std::stable_sort(cand.begin(), cand.end(), [](const Cand& a, const Cand& b) { return a.cost > b.cost; });
    typedef std::pair<int64_t, int> Load;                  // (assigned cost, CTA)
    std::priority_queue<Load, std::vector<Load>, std::greater<Load>> heap;
    for (int c = 0; c < grid; ++c) heap.push({0, c});
    std::vector<std::vector<StreamItem>> lists((size_t)grid);
    for (const Cand& cd : cand) {
        Load l = heap.top();
        heap.pop();
        lists[(size_t)l.second].push_back({cd.prob, cd.blk});
        heap.push({l.first + cd.cost, l.second});
    }
    int32_t* first = reinterpret_cast<int32_t*>(h_table + L.off_first);
    StreamItem* out_items = reinterpret_cast<StreamItem*>(h_table + L.off_items);
    int pos = 0;
    for (int c = 0; c < grid; ++c) {
        first[c] = pos;
        // within a CTA keep the layers in the order they were given: neighbouring CTAs then stream neighbouring rows
        std::stable_sort(lists[(size_t)c].begin(), lists[(size_t)c].end(),
                         [](const StreamItem& a, const StreamItem& b) { return a.prob != b.prob ? a.prob < b.prob : a.blk < b.blk; });
        for (const StreamItem& it : lists[(size_t)c]) out_items[pos++] = it;
    }
    first[grid] = pos;
    *grid_out = grid;
    *smem_out = H->smem_bytes;
    return true;
}

cudaError_t launch_stream(const uint8_t* d_table, int grid, uint32_t smem_bytes, cudaStream_t st)
{
    static bool attr_set[kMaxDevices] = {};
    if (!ensure_smem_attr(reinterpret_cast<const void*>(stream_kernel), kStreamSmem, attr_set)) return cudaErrorUnknown;
    stream_kernel<<<grid, kStreamThreads, smem_bytes, st>>>(d_table);
    return cudaGetLastError();
}

}  // namespace rmsmp
