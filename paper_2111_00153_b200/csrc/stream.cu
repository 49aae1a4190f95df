// Grouped weight-streaming kernel: many small-batch linear layers (up to 256 tokens each) in ONE
// launch on the tensor cores.
//
// With a handful of tokens a layer is bound by reading its packed weights once, and the only
// per-weight work is turning 4-bit codes into int8 operands.  One persistent CTA per SM walks its
// own list of work items; an item is one block of 128 ORIGINAL rows of one layer (the three runs
// of the packed buffer that hold those rows), the whole reduction, all tokens.  Per item the
// reduction is cut into stages of two k-blocks (256 codes).  Warp roles:
//   warp 0       producer.  Per stage: the packed codes of the item's rows as 16-row TMA boxes,
//                one lane per box, into a raw ring (4-bit rows bring 128 bytes per stage, 8-bit
//                rows 256); the activation codes of the two k-blocks as two swizzled boxes
//                [n_pad tokens][128 codes] (rows beyond a layer's token count read zeros).
//   warp 1       allocates tensor memory and issues tcgen05.mma kind::i8 (M = 128 rows, N = n_pad
//                tokens), eight instructions per stage; accumulators alternate between two
//                tensor-memory buffers so that an item's output overlaps the next item's stream.
//   warps 2-17   expanders: thread <-> (row slot, 16-byte chunk); raw codes -> int8 in registers ->
//                the K-major 128-byte-swizzled A tiles, each row at its ORIGINAL index, so the
//                accumulator lanes are in original row order and the output is coalesced.
//   warps 18-21  epilogue: tcgen05.ld, undo the x16 of Fixed-4 rows, scale by wstep * act_step,
//                direct coalesced stores (one token's 32 rows per warp instruction).
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

constexpr int kExpWarps = 16;
constexpr int kEpiWarps = 4;
constexpr int kStreamThreads = 32 * (2 + kExpWarps + kEpiWarps);      // 704
constexpr int kATile = kBlockRows * 128;                              // 16 KB: one expanded k-block
constexpr int kAStage = 2 * kATile;                                   // two k-blocks per stage
constexpr int kBoxRows = 16;                                          // rows per raw weight box
constexpr int kRingMax = 8;
constexpr int kStreamSmem = 232448 - 1024;
constexpr uint32_t kPlanMagic = 0x53545247u;                          // "STRG"

// One layer of the launch as the kernel sees it (device table, 128-byte aligned: it starts with
// the tensor maps).
struct alignas(128) StreamProblem {
    CUtensorMap q4, q8, act;        // packed 4-bit rows, packed 8-bit rows, activation codes [N][ld_act]
    const int32_t* perm;
    const float* wstep;
    const uint8_t* kind;
    const int32_t* blocks;
    float* out;
    int32_t* acc;
    uint32_t* status;
    int64_t ld_out;
    float act_step;
    int32_t M, N, nP, nF4, nkb, out_mn, pad0;
};
static_assert(sizeof(StreamProblem) % 128 == 0, "tensor maps stay 128-byte aligned in the array");

struct StreamItem { int32_t prob, blk; };

struct StreamHeader {               // first 128 bytes of the table
    uint32_t magic;
    int32_t nprob, nitems, grid;
    int32_t n_pad, nR, nA, nB;
    uint32_t raw_bytes, b_bytes, idesc, smem_bytes;
    uint32_t off_first, off_items, off_probs, bytes;
    uint32_t pad[16];
};
static_assert(sizeof(StreamHeader) == 128, "header is 128 bytes");

__device__ __forceinline__ int ceil_box(int n) { return (n + kBoxRows - 1) / kBoxRows * kBoxRows; }

struct BlockRuns { int p0, nP, f0, nF, e0, nE; };
__device__ __forceinline__ BlockRuns load_runs(const StreamProblem* P, int blk)
{
    const int4 b0 = __ldg(reinterpret_cast<const int4*>(P->blocks + 8 * blk));
    const int2 b1 = __ldg(reinterpret_cast<const int2*>(P->blocks + 8 * blk + 4));
    BlockRuns b;
    b.p0 = b0.x; b.nP = b0.y; b.f0 = b0.z; b.nF = b0.w; b.e0 = b1.x; b.nE = b1.y;
    return b;
}

// What an expander thread knows about one of its two rows of an item: bits 0-15 byte offset of its
// chunk inside a raw stage, bits 16-26 (in 16-byte units) offset of its first destination chunk
// inside an A stage, bits 30-31 kind (3: no such row).  c = 16-byte chunk index 0..7 of the thread.
__device__ __forceinline__ uint32_t stream_meta(const StreamProblem* P, int blk, int slot, int c)
{
    if (P == nullptr) return 3u << 30;
    const BlockRuns b = load_runs(P, blk);
    int kind, packed, raw;
    if (slot < b.nP) {
        kind = kPoT4; packed = b.p0 + slot; raw = slot * 128 + c * 16;
    } else if (slot < b.nP + b.nF) {
        kind = kFixed4; packed = P->nP + b.f0 + (slot - b.nP);
        raw = (ceil_box(b.nP) + slot - b.nP) * 128 + c * 16;
    } else if (slot < b.nP + b.nF + b.nE) {
        kind = kFixed8; packed = P->nP + P->nF4 + b.e0 + (slot - b.nP - b.nF);
        raw = (ceil_box(b.nP) + ceil_box(b.nF)) * 128 + (slot - b.nP - b.nF) * 256 + c * 16;
    } else {
        return 3u << 30;
    }
    const int row = __ldg(P->perm + packed) - blk * kBlockRows;
    uint32_t aoff;
    if (kind == kFixed8) {
        aoff = (uint32_t)row * 128u + ((uint32_t)(c ^ (row & 7)) << 4);                           // tile 0; tile 1 = + kATile
    } else {
        aoff = (uint32_t)(c >> 2) * kATile + (uint32_t)row * 128u + ((uint32_t)((2 * (c & 3)) ^ (row & 7)) << 4);
        if (c >= 4) aoff ^= 16u;          // the two halves in the other order: keeps a quarter-warp's stores on distinct banks
    }
    return (uint32_t)raw | ((aoff >> 4) << 16) | ((uint32_t)kind << 30);
}

__device__ __forceinline__ void lds128(uint32_t addr, uint32_t (&w)[4])
{
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// One task: a 16-byte raw chunk (32 four-bit codes, or 16 + 16 eight-bit codes of the two k-blocks)
// becomes two 16-byte chunks of expanded int8 values.
__device__ __forceinline__ void stream_expand(uint32_t meta, uint32_t raw_stage, uint32_t a_stage, bool upper)
{
    const uint32_t kind = meta >> 30;
    const uint32_t src = raw_stage + (meta & 0xFFFFu);
    const uint32_t dst = a_stage + (((meta >> 16) & 0x7FFu) << 4);
    if (kind == kFixed8) {
        uint32_t lo[4], hi[4];
        lds128(src, lo);
        lds128(src + 128, hi);
        sts128(dst, lo[0], lo[1], lo[2], lo[3]);
        sts128(dst + kATile, hi[0], hi[1], hi[2], hi[3]);
        return;
    }
    uint32_t r[4];
    lds128(src, r);
    const uint4 c = make_uint4(r[0], r[1], r[2], r[3]);
    uint32_t w[8];
    if (kind == kPoT4) expand_pot_chunk(c, w); else expand_fixed4_chunk_x16(c, w);
    // `dst` holds codes 0..15 of the chunk (or, for the upper four chunks, 16..31 first: see stream_meta)
    if (!upper) {
        sts128(dst, w[0], w[1], w[2], w[3]);
        sts128(dst ^ 16u, w[4], w[5], w[6], w[7]);
    } else {
        sts128(dst, w[4], w[5], w[6], w[7]);
        sts128(dst ^ 16u, w[0], w[1], w[2], w[3]);
    }
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
    const int n_pad = H->n_pad, nR = H->nR, nA = H->nA, nB = H->nB;
    const uint32_t raw_bytes = H->raw_bytes, b_bytes = H->b_bytes, idesc = H->idesc;
    const uint32_t b_sub = (uint32_t)n_pad * 128u;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sA = smem_base;
    const uint32_t sB = sA + nA * kAStage;
    const uint32_t sRaw = sB + nB * b_bytes;
    const uint32_t sBar = sRaw + nR * raw_bytes;
    const uint32_t bar_fullA = sBar, bar_emptyA = sBar + 8 * kRingMax;
    const uint32_t bar_fullB = sBar + 16 * kRingMax, bar_emptyB = sBar + 24 * kRingMax;
    const uint32_t bar_fullR = sBar + 32 * kRingMax, bar_emptyR = sBar + 40 * kRingMax;
    const uint32_t bar_tfull = sBar + 48 * kRingMax, bar_tempty = bar_tfull + 16;
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kRingMax; ++s) {
            mbar_init(bar_fullA + 8 * s, kExpWarps);     // one arrival per expander warp
            mbar_init(bar_emptyA + 8 * s, 1);            // tcgen05.commit
            mbar_init(bar_fullB + 8 * s, 1);             // producer (+ transaction bytes)
            mbar_init(bar_emptyB + 8 * s, 1);            // tcgen05.commit
            mbar_init(bar_fullR + 8 * s, 1);             // producer (+ transaction bytes)
            mbar_init(bar_emptyR + 8 * s, kExpWarps);    // one arrival per expander warp
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_tfull + 8 * b, 1);             // tcgen05.commit
            mbar_init(bar_tempty + 8 * b, kEpiWarps);    // one arrival per epilogue warp
        }
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
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

    if (warp == 0) {
        // ---------------------------------------------------------- producer
        uint32_t sr = 0, phR = 0, sb = 0, phB = 0;
        bool ok = true;
        int prev_prob = -1;
        for (int it = it0; it < it1 && ok; ++it) {
            const StreamItem item = items[it];
            const StreamProblem* P = probs + item.prob;
            last_status = P->status;
            const BlockRuns br = load_runs(P, item.blk);
            const int nbP = ceil_box(br.nP) / kBoxRows, nbF = ceil_box(br.nF) / kBoxRows, nbE = ceil_box(br.nE) / kBoxRows;
            const uint32_t raw_tx = (uint32_t)(nbP + nbF) * (kBoxRows * 128) + (uint32_t)nbE * (kBoxRows * 256);
            const CUtensorMap* my_map = nullptr;
            int my_row = 0, my_x8 = 0;
            uint32_t my_dst = 0;
            if (lane < nbP) { my_map = &P->q4; my_row = br.p0 + lane * kBoxRows; my_dst = lane * (kBoxRows * 128); }
            else if (lane < nbP + nbF) { my_map = &P->q4; my_row = P->nP + br.f0 + (lane - nbP) * kBoxRows; my_dst = lane * (kBoxRows * 128); }
            else if (lane < nbP + nbF + nbE) {
                my_map = &P->q8; my_x8 = 1; my_row = br.e0 + (lane - nbP - nbF) * kBoxRows;
                my_dst = (nbP + nbF) * (kBoxRows * 128) + (lane - nbP - nbF) * (kBoxRows * 256);
            }
            if (item.prob != prev_prob) {
                // the maps were written to the table by an earlier kernel: order this thread's use of them after that
                if (my_map) tensormap_acquire(my_map);
                if (lane == 0) tensormap_acquire(&P->act);
                prev_prob = item.prob;
            }
            const int nkb = P->nkb, npairs = (nkb + 1) >> 1;
            for (int kp = 0; kp < npairs; ++kp) {
                if (!mbar_wait_warp(bar_emptyR + 8 * sr, phR ^ 1, abort_flag)) { ok = false; break; }
                const uint32_t rbar = bar_fullR + 8 * sr;
                if (lane == 0) mbar_arrive_expect_tx(rbar, raw_tx);
                __syncwarp();
                if (my_map) tma_load_2d(sRaw + sr * raw_bytes + my_dst, my_map, rbar, my_x8 ? kp * 256 : kp * 128, my_row);
                if (++sr == (uint32_t)nR) { sr = 0; phR ^= 1; }
                if (!mbar_wait_warp(bar_emptyB + 8 * sb, phB ^ 1, abort_flag)) { ok = false; break; }
                if (lane == 0) {
                    const int nsub = (2 * kp + 1 < nkb) ? 2 : 1;
                    const uint32_t bbar = bar_fullB + 8 * sb;
                    mbar_arrive_expect_tx(bbar, (uint32_t)nsub * b_sub);
                    tma_load_2d(sB + sb * b_bytes, &P->act, bbar, kp * 256, 0);
                    if (nsub == 2) tma_load_2d(sB + sb * b_bytes + b_sub, &P->act, bbar, kp * 256 + 128, 0);
                }
                if (++sb == (uint32_t)nB) { sb = 0; phB ^= 1; }
            }
        }
        if (!ok && lane == 0) {
            for (int i = 0; i < 200; ++i) __nanosleep(1000);   // let copies in flight land before the CTA's memory is released
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------- MMA issuer (lane 0 issues; the warp walks in step)
        const bool issuer = (lane == 0);
        uint32_t sa = 0, phA = 0, sb = 0, phB = 0, n = 0;
        const uint64_t desc_a0 = smem_desc_kmajor(sA, 128), desc_b0 = smem_desc_kmajor(sB, 128);
        const uint32_t a_lo0 = (uint32_t)desc_a0, b_lo0 = (uint32_t)desc_b0, desc_hi = (uint32_t)(desc_a0 >> 32);
        bool ok = true;
        for (int it = it0; it < it1 && ok && !*abort_flag; ++it, ++n) {
            const StreamItem item = items[it];
            const StreamProblem* P = probs + item.prob;
            last_status = P->status;
            const int nkb = P->nkb, npairs = (nkb + 1) >> 1;
            const uint32_t ab = n & 1;
            if (!mbar_wait(bar_tempty + 8 * ab, ((n >> 1) & 1) ^ 1, abort_flag)) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + ab * 256;
            for (int kp = 0; kp < npairs; ++kp) {
                if (!mbar_wait(bar_fullB + 8 * sb, phB, abort_flag) || !mbar_wait(bar_fullA + 8 * sa, phA, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t a_lo = a_lo0 + sa * (kAStage >> 4), b_lo = b_lo0 + sb * (b_bytes >> 4);
                if (issuer) {
                    mma_i8_halves(d_tmem, a_lo, b_lo, desc_hi, idesc, kp ? 1u : 0u);
                    mma_i8_halves(d_tmem, a_lo + 2, b_lo + 2, desc_hi, idesc, 1u);
                    mma_i8_halves(d_tmem, a_lo + 4, b_lo + 4, desc_hi, idesc, 1u);
                    mma_i8_halves(d_tmem, a_lo + 6, b_lo + 6, desc_hi, idesc, 1u);
                    if (2 * kp + 1 < nkb) {
                        const uint32_t a1 = a_lo + (kATile >> 4), b1 = b_lo + (b_sub >> 4);
                        mma_i8_halves(d_tmem, a1, b1, desc_hi, idesc, 1u);
                        mma_i8_halves(d_tmem, a1 + 2, b1 + 2, desc_hi, idesc, 1u);
                        mma_i8_halves(d_tmem, a1 + 4, b1 + 4, desc_hi, idesc, 1u);
                        mma_i8_halves(d_tmem, a1 + 6, b1 + 6, desc_hi, idesc, 1u);
                    }
                    mma_commit(bar_emptyA + 8 * sa);
                    mma_commit(bar_emptyB + 8 * sb);
                }
                if (++sa == (uint32_t)nA) { sa = 0; phA ^= 1; }
                if (++sb == (uint32_t)nB) { sb = 0; phB ^= 1; }
            }
            if (!ok) break;
            if (issuer) mma_commit(bar_tfull + 8 * ab);
        }
    } else if (warp < 2 + kExpWarps) {
        // ---------------------------------------------------------- expanders
        const int et = (warp - 2) * 32 + lane;           // 0..511
        const int c = et & 7;                            // 16-byte chunk of a row's raw bytes in a stage
        const int slot0 = et >> 3;                       // row slots slot0 and slot0 + 64 of the item's sorted order
        const bool upper = c >= 4;
        uint32_t sa = 0, phA = 0, sr = 0, phR = 0;
        uint32_t cur[2], nxt[2];
        auto meta_of = [&](int it, int slot) -> uint32_t {
            if (it >= it1) return 3u << 30;
            const StreamItem item = items[it];
            return stream_meta(probs + item.prob, item.blk, slot, c);
        };
        cur[0] = meta_of(it0, slot0); cur[1] = meta_of(it0, slot0 + 64);
        bool ok = true;
        for (int it = it0; it < it1 && ok; ++it) {
            const StreamItem item = items[it];
            const StreamProblem* P = probs + item.prob;
            last_status = P->status;
            const int npairs = (P->nkb + 1) >> 1;
            nxt[0] = meta_of(it + 1, slot0); nxt[1] = meta_of(it + 1, slot0 + 64);     // in flight during this item
            for (int kp = 0; kp < npairs; ++kp) {
                if (!mbar_wait_warp(bar_fullR + 8 * sr, phR, abort_flag) ||
                    !mbar_wait_warp(bar_emptyA + 8 * sa, phA ^ 1, abort_flag)) { ok = false; break; }
                const uint32_t rs = sRaw + sr * raw_bytes, as = sA + sa * kAStage;
                if ((cur[0] >> 30) != 3u) stream_expand(cur[0], rs, as, upper);
                if ((cur[1] >> 30) != 3u) stream_expand(cur[1], rs, as, upper);
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(bar_fullA + 8 * sa);
                    mbar_arrive(bar_emptyR + 8 * sr);
                }
                if (++sa == (uint32_t)nA) { sa = 0; phA ^= 1; }
                if (++sr == (uint32_t)nR) { sr = 0; phR ^= 1; }
            }
            cur[0] = nxt[0]; cur[1] = nxt[1];
        }
    } else {
        // ---------------------------------------------------------- epilogue
        const int quarter = warp & 3;                    // tensor-memory lanes this warp may read
        uint32_t n = 0;
        bool alive = true;
        // this warp's row of the first item: scale and Fixed-4 shift, fetched ahead of the accumulator
        auto row_info = [&](int it, float& scale, int& shift, int& m, bool& row_ok) {
            scale = 0.f; shift = 0; m = 0; row_ok = false;
            if (it >= it1) return;
            const StreamItem item = items[it];
            const StreamProblem* P = probs + item.prob;
            m = item.blk * kBlockRows + quarter * 32 + lane;
            row_ok = m < P->M;
            if (row_ok) {
                scale = __fmul_rn(__ldg(P->wstep + m), P->act_step);
                shift = (__ldg(P->kind + m) == kFixed4) ? 4 : 0;     // expanders store Fixed-4 codes as 16 * value
            }
        };
        float scale, scale_n; int shift, shift_n, m, m_n; bool row_ok, row_ok_n;
        row_info(it0, scale, shift, m, row_ok);
        for (int it = it0; it < it1 && alive; ++it, ++n) {
            const StreamItem item = items[it];
            const StreamProblem* P = probs + item.prob;
            last_status = P->status;
            row_info(it + 1, scale_n, shift_n, m_n, row_ok_n);
            const uint32_t ab = n & 1;
            if (!mbar_wait_warp(bar_tfull + 8 * ab, (n >> 1) & 1, abort_flag)) { alive = false; break; }
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + ab * 256;
            const int N = P->N;
            const int nchunks = (N + 31) >> 5;
            float* const out = P->out;
            int32_t* const acc = P->acc;
            const int64_t ld = P->ld_out;
            const bool out_mn = P->out_mn != 0;
            for (int ch = 0; ch < nchunks; ++ch) {
                uint32_t v[32];
                tmem_ld_issue(taddr + ch * 32, v);
                tmem_ld_wait(v);
                if (ch == nchunks - 1) {
                    // every accumulator of this item is in registers: hand the buffer back
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_tempty + 8 * ab);
                }
                if (!row_ok) continue;
                const int jmax = min(32, N - ch * 32);
                if (!out_mn) {
                    float* o = out + (int64_t)(ch * 32) * ld + m;
                    int32_t* oa = acc ? acc + (int64_t)(ch * 32) * ld + m : nullptr;
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        if (j < jmax) {
                            const int a = (int)v[j] >> shift;
                            o[(int64_t)j * ld] = __fmul_rn(__int2float_rn(a), scale);
                            if (oa) oa[(int64_t)j * ld] = a;
                        }
                    }
                } else {
                    float* o = out + (int64_t)m * ld + ch * 32;
                    int32_t* oa = acc ? acc + (int64_t)m * ld + ch * 32 : nullptr;
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        if (j < jmax) {
                            const int a = (int)v[j] >> shift;
                            o[j] = __fmul_rn(__int2float_rn(a), scale);
                            if (oa) oa[j] = a;
                        }
                    }
                }
            }
            scale = scale_n; shift = shift_n; m = m_n; row_ok = row_ok_n;
        }
    }

    // ---------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
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
    if (p.kh != 1 || p.kw != 1 || p.N < 1 || p.N > 256) return false;
    if (p.pix_pitch % 16 != 0 || (reinterpret_cast<uintptr_t>(p.act) & 15) != 0) return false;
    if (p.raw_stage_bytes <= 0 || 2 * (int64_t)p.raw_stage_bytes > 64 * 1024) return false;
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
    int raw1 = 0;
    for (int i = 0; i < count; ++i) {
        nitems += probs[i].nblocks;
        maxN = std::max<int64_t>(maxN, probs[i].N);
        raw1 = std::max(raw1, probs[i].raw_stage_bytes);
    }
    if (nitems >= (1ll << 30)) return false;
    const int grid = (int)std::min<int64_t>(sms, nitems);
    const Layout L = table_layout(count, (int)nitems, grid);
    if (L.bytes > table_bytes) return false;
    memset(h_table, 0, L.bytes);
    StreamHeader* H = reinterpret_cast<StreamHeader*>(h_table);
    H->magic = kPlanMagic; H->nprob = count; H->nitems = (int32_t)nitems; H->grid = grid;
    H->n_pad = std::max(16, (int)((maxN + 15) / 16 * 16));
    H->raw_bytes = (uint32_t)up((size_t)2 * raw1, 1024);
    H->b_bytes = (uint32_t)(2 * H->n_pad * 128);
    // shared-memory budget: two expanded stages; up to four activation stages (a third of what is left at
    // most); everything else is the raw ring, i.e. what is in flight from HBM
    const int64_t avail = kStreamSmem - 1024 - 64 * kRingMax;
    H->nA = 2;
    int64_t left = avail - (int64_t)H->nA * kAStage;
    H->nB = (int)std::min<int64_t>(4, std::max<int64_t>(2, left / 3 / H->b_bytes));
    left -= (int64_t)H->nB * H->b_bytes;
    H->nR = (int)std::min<int64_t>(kRingMax, left / H->raw_bytes);
    if (H->nR < 2) return false;
    H->smem_bytes = (uint32_t)(H->nA * kAStage + H->nB * H->b_bytes + H->nR * H->raw_bytes + 1024 + 64 * kRingMax);
    // kind::i8: int32 accumulate, signed 8-bit A and B, both K-major, N/8 at bit 17, M/16 at bit 24
    H->idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(H->n_pad >> 3) << 17) | ((uint32_t)(kBlockRows >> 4) << 24);
    H->off_first = (uint32_t)L.off_first; H->off_items = (uint32_t)L.off_items; H->off_probs = (uint32_t)L.off_probs;
    H->bytes = (uint32_t)L.bytes;

    // problems and their tensor maps
    StreamProblem* sp = reinterpret_cast<StreamProblem*>(h_table + L.off_probs);
    for (int i = 0; i < count; ++i) {
        const Problem& p = probs[i];
        StreamProblem& q = sp[i];
        auto make_w = [&](CUtensorMap* m, const uint8_t* base, int rows, int pitch, int box_bytes) -> bool {
            if (rows <= 0) return true;
            const cuuint64_t gd[2] = {(cuuint64_t)pitch, (cuuint64_t)rows};
            const cuuint64_t gs[1] = {(cuuint64_t)pitch};
            const cuuint32_t bx[2] = {(cuuint32_t)box_bytes, (cuuint32_t)kBoxRows};
            const cuuint32_t es[2] = {1, 1};
            return enc(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(base), gd, gs, bx, es,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
        };
        if (!make_w(&q.q4, p.q4, p.nP + p.nF4, p.Kp / 2, 128) || !make_w(&q.q8, p.q8, p.n8, p.Kp, 256)) return false;
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
