// Tensor-core variant of the contraction for sm_100a.
//
// One persistent CTA per SM walks over output tiles of 128 weight rows x up to 256 pixels; the
// reduction is cut into k-blocks of 128 codes.  Warp roles:
//   warp 0      TMA producer.  Per k-block it fetches (a) the activation-code tile (the B
//               operand): one 4-D box into 128-byte-swizzled shared memory -- for a convolution
//               the box is the window of input pixels one filter tap needs, zero fill outside the
//               image being the padding, so no im2col buffer exists anywhere; (b) the packed
//               4-bit / 8-bit weight codes of the tile's rows, as 16-row boxes, into a raw ring.
//   warp 1      allocates tensor memory and issues tcgen05.mma (kind::i8, int32 accumulators in
//               tensor memory, two 256-column buffers: tile i+1 is computed while tile i is
//               written out).
//   warps 2-9   expanders, two groups of four warps that take alternate k-blocks: read the raw
//               codes from shared memory, expand them to int8 in registers and store them in the
//               K-major 128-byte-swizzled layout the MMA reads (the A operand).  Rows arrive
//               group by group (PoT, Fixed-4, Fixed-8) but are written to the row of their ORIGINAL
//               index, so accumulator lanes are in original row order and the output needs no
//               scatter through the permutation.
//   warps 10-13 epilogue, one per tensor-memory quarter (in workspace mode the expander warps
//               have nothing to expand and join the epilogue, three warps per quarter): tcgen05.ld (next chunk in flight while
//               the current one is processed), undo the x16 of Fixed-4 rows, convert, scale by
//               wstep*act_step, stage 32 pixels x 32 rows in a private double buffer and write it
//               with a bulk tensor store.
// Every wait on an mbarrier is bounded; when one runs out the kernel records
// RMSMP_ERR_TIMEOUT in the packed buffer's status word, all roles leave their loops, tensor
// memory is freed and the kernel returns.
#include <cuda.h>
#include <cstring>
#include "common.cuh"
#include "decode.cuh"
#include "actq.cuh"
#include "ptx.cuh"
#include "tmap.cuh"

namespace rmsmp {

namespace {

constexpr int kTileN = 256;                      // pixels per tile (max) = TMEM columns per buffer
constexpr int kABytes = kBlockRows * 128;        // 16 KB: 128 rows x 128 B (one k-block)
constexpr int kBBytes = kTileN * 128;            // 32 KB
constexpr int kGroups = 2;                       // expander groups taking alternate k-blocks
constexpr int kNumExpWarps = 4 * kGroups;
constexpr int kNumEpiWarps = 4;
constexpr int kThreads = 32 * (2 + kNumExpWarps + kNumEpiWarps);
constexpr int kWarpStage = 32 * 32 * 4;          // 4 KB: 32 pixels x 32 rows of fp32/int32
constexpr int kRawBoxRows = 16;                  // rows per raw weight box
constexpr int kMaxRing = 8;
constexpr int kSmemLimit = 232448 - 1024;        // 227 KB per CTA less room for the static variables

struct TensorCfg {
    int tb, th;            // images / output rows per tile
    int npix;              // pixels per full tile = tb*th*Wo
    int n_mma;             // npix rounded up to 16
    int tiles_per_image;   // Ho/th when tb == 1 and th < Ho, else 0
    int64_t ntiles_n;
    int64_t ntiles;        // ntiles_n * nblocks
    int cpt;               // 128-channel chunks per tap
    int nkb;               // k-blocks per tile = taps * cpt
    int last_ksteps;       // 32-code steps in the last chunk of a tap
    uint32_t idesc;
    uint32_t tx_bytes;     // bytes one activation box brings
    int tma_store;         // 1: output chunks leave through shared memory and bulk tensor stores
    int tail_rows;         // npix % 32: height of the last chunk of a tile (0: none)
    int nA, nB, nR;        // ring depths: expanded weights, activations, raw weights
    uint32_t raw_bytes;    // one raw stage
    int out_bufs;          // staging buffers per epilogue warp (1 or 2)
    int pre;               // 1: the A operand comes expanded (int8) from a workspace, no expander work
    int dup;               // 1 (pre mode, M <= 64): rows 0..63 are loaded twice, into lanes 0..63 and 64..127, so that all
                           //    four tensor-memory quarters hold valid rows and every epilogue warp has work
    int epi_warps;         // epilogue warps: 4, or 12 in pre mode (the idle expander warps join)
    int bk;                // codes per k-block and bytes per operand row in shared memory: 128, or 64 (pre mode,
                           //    channel counts that would leave half of a 128-byte row empty)
    int a_bytes, b_bytes;  // one A / B stage
    int fill;              // 1 (resident weights, no workspace given): the CTA expands its row block from the packed codes
                           //    itself, once, instead of copying expanded weights in
    int ares;              // 1 (pre mode, one row block, small K): the expanded weights of all k-blocks are loaded once
                           //    per CTA and stay in shared memory; only activation boxes flow through a ring
    int m2;                // 1 (pre mode, even number of row blocks): a tile covers TWO row blocks.  Both use the same
                           //    activation stage, so a k-block brings 64 KB for eight MMAs instead of 48 KB for four;
                           //    the two accumulators take the two halves of tensor memory
    int nbt;               // row-block groups per pixel tile: nblocks, or nblocks / 2
    int tps;               // k-blocks per activation stage: 1, or 3 (resident weights, 64-byte k-blocks, 3-wide kernels):
                           //    one barrier round trip then covers a whole kernel row instead of a single tap
    int b_sub;             // bytes of one k-block inside an activation stage
    int colshift;          // 1 (with tps == 3; 3x3, stride 1, tiles of whole output rows of one image, W % 8 == 0): an activation
                           //    stage holds the th + 2 input rows the tile needs at ONE column shift j, fetched once; the
                           //    taps (0..2, j) read it at row offsets of W pixels (whole swizzle atoms).  The copy engine
                           //    then moves 3 (th + 2) rows per tile instead of 9 th
    uint32_t smem_bytes;
};

struct Maps {
    CUtensorMap act[4];                                // [B][H][W][Cin] activation codes; stride 2: one map per row/column parity
    CUtensorMap q4, q8;                                // packed weight regions
    CUtensorMap wexp;                                  // [M][Kp] int8 weights expanded beforehand (pre mode); 64-row box when dup
    CUtensorMap out_full, out_tail, acc_full, acc_tail;   // bulk stores: 32-row and tail chunks
    CUtensorMap rq_full, rq_tail;                       // re-quantized codes: 32 pixels x 32 code bytes, and the tail
};

// ------------------------------------------------------------------ per-tile row bookkeeping

// Rows of one 128-row block inside the three groups of the packed buffer.
struct BlockInfo {
    int p0, nP, f0, nF, e0, nE;
};
__device__ __forceinline__ BlockInfo load_block(const Problem& p, int blk)
{
    const int4 b0 = __ldg(reinterpret_cast<const int4*>(p.blocks + 8 * blk));
    const int2 b1 = __ldg(reinterpret_cast<const int2*>(p.blocks + 8 * blk + 4));
    BlockInfo b;
    b.p0 = b0.x; b.nP = b0.y; b.f0 = b0.z; b.nF = b0.w; b.e0 = b1.x; b.nE = b1.y;
    return b;
}
__device__ __forceinline__ int ceil_box(int n) { return (n + kRawBoxRows - 1) / kRawBoxRows * kRawBoxRows; }

// What an expander thread knows about one of its rows in a tile, in one word:
// bits 0-15 byte offset of its 32 codes inside a raw stage, bits 16-29 byte offset of its first
// 16-byte chunk inside an A stage (the second chunk is that offset ^ 16), bits 30-31 kind (3: none).
__device__ __forceinline__ uint32_t make_meta(const Problem& p, int64_t tile, int slot, int q)
{
    if (tile < 0) return 3u << 30;
    const int blk = (int)(tile % p.nblocks);
    const BlockInfo b = load_block(p, blk);
    int kind, packed, raw;
    if (slot < b.nP) {
        kind = kPoT4; packed = b.p0 + slot; raw = slot * 64 + q * 16;
    } else if (slot < b.nP + b.nF) {
        kind = kFixed4; packed = p.nP + b.f0 + (slot - b.nP);
        raw = (ceil_box(b.nP) + slot - b.nP) * 64 + q * 16;
    } else if (slot < b.nP + b.nF + b.nE) {
        kind = kFixed8; packed = p.nP + p.nF4 + b.e0 + (slot - b.nP - b.nF);
        raw = (ceil_box(b.nP) + ceil_box(b.nF)) * 64 + (slot - b.nP - b.nF) * 128 + q * 32;
    } else {
        return 3u << 30;
    }
    const int row = __ldg(p.perm + packed) - blk * kBlockRows;
    const uint32_t aoff = (uint32_t)row * 128u + ((uint32_t)((2 * q) ^ (row & 7)) << 4);
    return (uint32_t)raw | (aoff << 16) | ((uint32_t)kind << 30);
}

// Expand one task: 32 codes from the raw stage to two 16-byte chunks of the A stage.
__device__ __forceinline__ void expand_task(uint32_t meta, uint32_t raw_stage, uint32_t a_stage)
{
    const uint32_t kind = meta >> 30;
    const uint32_t src = raw_stage + (meta & 0xFFFFu);
    const uint32_t dst = a_stage + ((meta >> 16) & 0x3FFFu);
    uint32_t w[8];
    if (kind == kFixed8) {
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(src) : "memory");
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7]) : "r"(src + 16) : "memory");
    } else {
        uint4 c;
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(c.x), "=r"(c.y), "=r"(c.z), "=r"(c.w) : "r"(src) : "memory");
        if (kind == kPoT4) expand_pot_chunk(c, w); else expand_fixed4_chunk_x16(c, w);
    }
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst ^ 16u), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7]) : "memory");
}

// Resident weights without a workspace: every thread of the CTA expands 16-code granules of the row block
// from the packed codes (exact int8 values, as expand_kernel writes them) straight into the resident stages,
// at the place the bulk copy of an expanded [rows][bk] box would have put them: stage kb = (tap, channel
// chunk) holds codes [tap * Cp + chunk * bk, + bk) of every row, 16-byte units XOR-swizzled by the row
// (128-byte rows: unit ^ (row & 7); 64-byte rows: unit ^ ((row >> 1) & 3)), zeros beyond M and Kp; with
// duplicated rows (M <= 64) a second copy goes to lanes 64..127.
__device__ __forceinline__ void fill_resident_weights(const Problem& p, const TensorCfg& cfg, uint32_t sA, int tid, int nthreads)
{
    const int rows = cfg.dup ? kBlockRows / 2 : kBlockRows;
    const int gpr = cfg.bk >> 4;
    const int n4 = p.nP + p.nF4;
    // a few threads per row, each with every tpr-th granule of it: kind and place of the row are read once, and a
    // thread's loads are independent of one another
    const int tpr = nthreads / rows;
    const int r = tid / tpr, sub = tid - r * tpr;
    if (r < rows) {
        const bool have = r < p.M;
        const int kind = have ? (int)p.kind[r] : kFixed8;
        const int slot = have ? p.slot[r] : 0;
        const uint8_t* src = (kind == kFixed8) ? p.q8 + (size_t)(have ? slot - n4 : 0) * p.Kp : p.q4 + (size_t)slot * (p.Kp >> 1);
        const uint32_t phase = (cfg.bk == 128) ? (uint32_t)(r & 7) : (uint32_t)((r >> 1) & 3);
        const uint32_t row_base = sA + (uint32_t)r * (uint32_t)cfg.bk;
        const int gtot = cfg.nkb * gpr;
#pragma unroll 4
        for (int g = sub; g < gtot; g += tpr) {
            const int kb = g / gpr, q = g - kb * gpr;
            const int tap = kb / cfg.cpt, cc = kb - tap * cfg.cpt;
            const int k = tap * p.Cp + cc * cfg.bk + q * 16;
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (have && k < p.Kp) {
                if (kind == kFixed8) {
                    v = __ldg(reinterpret_cast<const uint4*>(src + k));
                } else {
                    const uint4 raw = __ldg(reinterpret_cast<const uint4*>(src + ((k >> 5) << 4)));
                    uint32_t w[8];
                    if (kind == kPoT4) {
                        expand_pot_chunk(raw, w);
                    } else {
                        expand_fixed4_chunk_x16(raw, w);
#pragma unroll
                        for (int j = 0; j < 8; ++j) {       // 16 * value -> value: shift every byte right by four, keeping its sign
                            const uint32_t x = w[j];
                            w[j] = ((x >> 4) & 0x0F0F0F0Fu) | (((x >> 7) & 0x01010101u) * 0xF0u);
                        }
                    }
                    const int h = (k >> 4) & 1;
                    v = h ? make_uint4(w[4], w[5], w[6], w[7]) : make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
            const uint32_t dst = row_base + (uint32_t)kb * (uint32_t)cfg.a_bytes + (((uint32_t)q ^ phase) << 4);
            // (no memory clobber: the loads of the next granules may move above these stores)
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w));
            if (cfg.dup)
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst + (uint32_t)(cfg.a_bytes / 2)), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w));
        }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // the MMAs read these bytes through the async proxy
}

// ------------------------------------------------------------------ the kernel

// kM2: a tile covers two row blocks (TensorCfg::m2), compiled separately so that the common form keeps its registers.
// kRQ: the epilogue writes the next layer's activation codes instead of fp32 (Problem::rq_codes).
// kMode: which of the kernel's forms this instantiation is (the host picks it from the plan): 0 codes expanded in
//        shared memory; 1 expanded weights from a workspace through the ring; 2 the same, weights resident in
//        shared memory; 3 resident weights and three taps per activation stage.  A compile-time constant so that
//        an instantiation carries only the code of its own form.
// kOut:  1 when the output is fp32 [N][M] through bulk stores without an accumulator dump (the common case): the
//        epilogue then carries only that path; 0 decides at run time.
template <int kM2, int kRQ, int kMode, int kOut>
__global__ void __launch_bounds__(kThreads, 1)
tensor_kernel(const Problem p, const TensorCfg cfg, const __grid_constant__ Maps maps)
{
    constexpr bool kPre = kMode != 0, kAres = kMode >= 2, kTps3 = kMode == 3;
    const bool use_tma_store = kOut ? true : (cfg.tma_store != 0);
    const bool out_mn = kOut ? false : (p.out_mn != 0);
    int32_t* const acc_out = kOut ? nullptr : p.acc;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sA = smem_base;
    const uint32_t sB = sA + cfg.nA * cfg.a_bytes;
    const uint32_t sRaw = sB + cfg.nB * cfg.b_bytes;
    const uint32_t sOut = sRaw + cfg.nR * cfg.raw_bytes;
    const uint32_t sBar = sOut + cfg.epi_warps * cfg.out_bufs * kWarpStage;
    // barriers, 8 bytes each
    const uint32_t bar_fullA = sBar, bar_emptyA = sBar + 8 * kMaxRing;
    const uint32_t bar_fullB = sBar + 16 * kMaxRing, bar_emptyB = sBar + 24 * kMaxRing;
    const uint32_t bar_fullR = sBar + 32 * kMaxRing, bar_emptyR = sBar + 40 * kMaxRing;
    const uint32_t bar_tfull = sBar + 48 * kMaxRing, bar_tempty = bar_tfull + 16;
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxRing; ++s) {
            mbar_init(bar_fullA + 8 * s, kPre ? 1 : 4);   // producer (+ bytes), or the four warps of one expander group
            mbar_init(bar_emptyA + 8 * s, 1);    // tcgen05.commit
            mbar_init(bar_fullB + 8 * s, 1);     // producer (+ transaction bytes)
            mbar_init(bar_emptyB + 8 * s, 1);    // tcgen05.commit
            mbar_init(bar_fullR + 8 * s, 1);     // producer (+ transaction bytes)
            mbar_init(bar_emptyR + 8 * s, 4);    // the four warps of one expander group
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_tfull + 8 * b, 1);                  // tcgen05.commit
            mbar_init(bar_tempty + 8 * b, cfg.epi_warps);     // one arrival per epilogue warp
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

    const int64_t first = blockIdx.x, step = gridDim.x;
    const int64_t my_tiles = (cfg.ntiles > first) ? (cfg.ntiles - first + step - 1) / step : 0;

    if (kAres && cfg.fill && warp != 0) {
        // every warp but the activation producer's (whose first copies go out meanwhile) expands the row block;
        // one of them then reports the resident weights to the MMA thread
        if (my_tiles > 0) fill_resident_weights(p, cfg, sA, (int)threadIdx.x - 32, kThreads - 32);
        asm volatile("bar.sync 1, %0;" ::"n"(kThreads - 32) : "memory");
        if (threadIdx.x == 32 && my_tiles > 0) mbar_arrive(bar_fullA);
    }

    // Workspace mode splits the producer: one thread can start a bulk tensor copy only every few
    // hundred cycles, so the activation boxes and the weight boxes are issued by two different warps.
    const bool pre_b_producer = kPre && warp == 0;
    const bool pre_a_producer = kPre && !kAres && warp == 2;
    if (pre_b_producer || pre_a_producer) {
        if (lane == 0) {
            if (pre_b_producer && kAres && my_tiles > 0 && !cfg.fill) {
                // resident weights: every k-block's rows, once
                mbar_arrive_expect_tx(bar_fullA, (uint32_t)(cfg.nkb * cfg.a_bytes));
                int tap = 0, cc = 0;
                for (int kb = 0; kb < cfg.nkb; ++kb) {
                    const int koff = tap * p.Cp + cc * cfg.bk;
                    const uint32_t dst = sA + kb * cfg.a_bytes;
                    tma_load_2d(dst, &maps.wexp, bar_fullA, koff, 0);
                    if (cfg.dup) tma_load_2d(dst + cfg.a_bytes / 2, &maps.wexp, bar_fullA, koff, 0);
                    if (++cc == cfg.cpt) { cc = 0; ++tap; }
                }
            }
            const uint32_t nring = pre_b_producer ? (uint32_t)cfg.nB : (uint32_t)cfg.nA;
            const uint32_t bar_e = pre_b_producer ? bar_emptyB : bar_emptyA;
            const uint32_t bar_f = pre_b_producer ? bar_fullB : bar_fullA;
            uint32_t s = 0, ph = 0;
            bool ok = true;
            for (int64_t tile = first; tile < cfg.ntiles && ok; tile += step) {
                const uint32_t nt = (uint32_t)tile / (uint32_t)cfg.nbt;
                const int blk = (int)((uint32_t)tile - nt * (uint32_t)cfg.nbt) << kM2;
                int b0, h0;
                if (cfg.tiles_per_image) {
                    b0 = (int)(nt / (uint32_t)cfg.tiles_per_image);
                    h0 = (int)(nt - (uint32_t)b0 * (uint32_t)cfg.tiles_per_image) * cfg.th;
                } else {
                    b0 = (int)nt * cfg.tb;
                    h0 = 0;
                }
                const int row_a = cfg.dup ? 0 : blk * kBlockRows;
                int tap = 0, cc = 0, ti = 0, tj = 0;
                for (int kb = 0; kb < cfg.nkb; ++kb) {
                    if (!mbar_wait(bar_e + 8 * s, ph ^ 1, abort_flag)) { ok = false; break; }
                    if (pre_b_producer && kTps3) {
                        if (cfg.colshift) {
                            // one stage = one column shift: the th + kh - 1 input rows the tile needs, fetched once
                            // and read by the kh taps of that column at row offsets (see TensorCfg::colshift)
                            mbar_arrive_expect_tx(bar_f + 8 * s, cfg.tx_bytes);
                            tma_load_4d(sB + s * cfg.b_bytes, &maps.act[0], bar_f + 8 * s, 0, ti - p.pad, h0 - p.pad, b0);
                        } else {
                            // one stage = the taps of one kernel row (one channel chunk per tap in this mode)
                            mbar_arrive_expect_tx(bar_f + 8 * s, cfg.tps * cfg.tx_bytes);
                            for (int t = 0; t < cfg.tps; ++t) {
                                const TapBox tb = tap_box(p, h0, ti, tj + t);
                                tma_load_4d(sB + s * cfg.b_bytes + t * cfg.b_sub, &maps.act[tb.map], bar_f + 8 * s, 0, tb.x, tb.y, b0);
                            }
                        }
                        ++ti;
                        kb += cfg.tps - 1;
                        if (++s == nring) { s = 0; ph ^= 1; }
                        continue;
                    }
                    if (pre_b_producer) {
                        mbar_arrive_expect_tx(bar_f + 8 * s, cfg.tx_bytes);
                        const TapBox tb = tap_box(p, h0, ti, tj);
                        tma_load_4d(sB + s * cfg.b_bytes, &maps.act[tb.map], bar_f + 8 * s, cc * cfg.bk, tb.x, tb.y, b0);
                    } else {
                        const int koff = tap * p.Cp + cc * cfg.bk;
                        mbar_arrive_expect_tx(bar_f + 8 * s, cfg.a_bytes);
                        tma_load_2d(sA + s * cfg.a_bytes, &maps.wexp, bar_f + 8 * s, koff, row_a);
                        if (cfg.dup) tma_load_2d(sA + s * cfg.a_bytes + cfg.a_bytes / 2, &maps.wexp, bar_f + 8 * s, koff, row_a);
                    }
                    if (++s == nring) { s = 0; ph ^= 1; }
                    if (++cc == cfg.cpt) { cc = 0; ++tap; if (++tj == p.kw) { tj = 0; ++ti; } }
                }
            }
            if (!ok) {
                for (int i = 0; i < 200; ++i) __nanosleep(1000);   // let copies in flight land
            }
        }
    } else if (warp == 0) {
        // ---------------------------------------------------------- TMA producer (shared-memory expansion mode)
        // The whole warp takes part: lane 0 waits on the barriers and fetches the activation box,
        // the weight boxes of a k-block are issued by one lane each.
        {
            uint32_t sb = 0, phB = 0, sr = 0, phR = 0;
            bool ok = true;
            if (kAres && lane == 0 && my_tiles > 0) {
                // resident weights: every k-block's rows, once
                mbar_arrive_expect_tx(bar_fullA, (uint32_t)(cfg.nkb * cfg.a_bytes));
                int tap = 0, cc = 0;
                for (int kb = 0; kb < cfg.nkb; ++kb) {
                    const int koff = tap * p.Cp + cc * cfg.bk;
                    const uint32_t dst = sA + kb * cfg.a_bytes;
                    if (cfg.dup) {
                        tma_load_2d(dst, &maps.wexp, bar_fullA, koff, 0);
                        tma_load_2d(dst + cfg.a_bytes / 2, &maps.wexp, bar_fullA, koff, 0);
                    } else {
                        tma_load_2d(dst, &maps.wexp, bar_fullA, koff, 0);
                    }
                    if (++cc == cfg.cpt) { cc = 0; ++tap; }
                }
            }
            for (int64_t tile = first; tile < cfg.ntiles && ok; tile += step) {
                const int blk = (int)(tile % p.nblocks);
                const int64_t nt = tile / p.nblocks;
                int b0, h0;
                if (cfg.tiles_per_image) { b0 = (int)(nt / cfg.tiles_per_image); h0 = (int)(nt % cfg.tiles_per_image) * cfg.th; }
                else { b0 = (int)(nt * cfg.tb); h0 = 0; }
                const BlockInfo bi = load_block(p, blk);
                const int nbP = ceil_box(bi.nP) / kRawBoxRows, nbF = ceil_box(bi.nF) / kRawBoxRows,
                          nbE = ceil_box(bi.nE) / kRawBoxRows;
                const uint32_t raw_tx = (uint32_t)(nbP + nbF) * (kRawBoxRows * 64) + (uint32_t)nbE * (kRawBoxRows * 128);
                // this lane's weight box (lanes beyond the box count have none)
                const CUtensorMap* my_map = nullptr;
                int my_row = 0, my_x8 = 0;           // my_x8: 1 if the box is in the 8-bit region
                uint32_t my_dst = 0;
                if (lane < nbP) { my_map = &maps.q4; my_row = bi.p0 + lane * kRawBoxRows; my_dst = lane * (kRawBoxRows * 64); }
                else if (lane < nbP + nbF) { my_map = &maps.q4; my_row = p.nP + bi.f0 + (lane - nbP) * kRawBoxRows; my_dst = lane * (kRawBoxRows * 64); }
                else if (lane < nbP + nbF + nbE) {
                    my_map = &maps.q8; my_x8 = 1; my_row = bi.e0 + (lane - nbP - nbF) * kRawBoxRows;
                    my_dst = (nbP + nbF) * (kRawBoxRows * 64) + (lane - nbP - nbF) * (kRawBoxRows * 128);
                }
                int tap = 0, cc = 0;
                for (int kb = 0; kb < cfg.nkb; ++kb) {
                    const int c0 = cc * cfg.bk, koff = tap * p.Cp + c0;
                    if (kAres) {
                        // weights are resident
                    } else if (kPre) {
                        // weights already expanded: one swizzled 128-row box straight into the A stage
                        if (!mbar_wait_warp(bar_emptyA + 8 * sr, phR ^ 1, abort_flag)) { ok = false; break; }
                        if (lane == 0) {
                            mbar_arrive_expect_tx(bar_fullA + 8 * sr, cfg.a_bytes);
                            if (cfg.dup) {
                                tma_load_2d(sA + sr * cfg.a_bytes, &maps.wexp, bar_fullA + 8 * sr, koff, 0);
                                tma_load_2d(sA + sr * cfg.a_bytes + cfg.a_bytes / 2, &maps.wexp, bar_fullA + 8 * sr, koff, 0);
                            } else {
                                tma_load_2d(sA + sr * cfg.a_bytes, &maps.wexp, bar_fullA + 8 * sr, koff, blk * kBlockRows);
                            }
                        }
                        if (++sr == (uint32_t)cfg.nA) { sr = 0; phR ^= 1; }
                    } else {
                        // packed weights of this tile's rows, group by group
                        if (!mbar_wait_warp(bar_emptyR + 8 * sr, phR ^ 1, abort_flag)) { ok = false; break; }
                        const uint32_t rbar = bar_fullR + 8 * sr;
                        if (lane == 0) mbar_arrive_expect_tx(rbar, raw_tx);
                        __syncwarp();
                        if (my_map) tma_load_2d(sRaw + sr * cfg.raw_bytes + my_dst, my_map, rbar, my_x8 ? koff : (koff >> 1), my_row);
                        if (++sr == (uint32_t)cfg.nR) { sr = 0; phR ^= 1; }
                    }
                    // activation codes
                    if (!mbar_wait_warp(bar_emptyB + 8 * sb, phB ^ 1, abort_flag)) { ok = false; break; }
                    if (lane == 0) {
                        const int ti = tap / p.kw, tj = tap - ti * p.kw;
                        mbar_arrive_expect_tx(bar_fullB + 8 * sb, cfg.tx_bytes);
                        const TapBox tb = tap_box(p, h0, ti, tj);
                        tma_load_4d(sB + sb * cfg.b_bytes, &maps.act[tb.map], bar_fullB + 8 * sb, c0, tb.x, tb.y, b0);
                    }
                    if (++sb == (uint32_t)cfg.nB) { sb = 0; phB ^= 1; }
                    if (++cc == cfg.cpt) { cc = 0; ++tap; }
                }
            }
            if (!ok && lane == 0) {
                // give copies already in flight time to land before the CTA's memory is released
                for (int i = 0; i < 200; ++i) __nanosleep(1000);
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------- MMA issuer
        // The whole warp walks the loops in step (so that ring positions and descriptors are
        // warp-uniform values); lane 0 alone issues the MMAs and commits.
        const bool issuer = (lane == 0);
        {
            uint32_t sa = 0, phA = 0, sb = 0, phB = 0, it = 0;
            const uint64_t desc_a0 = smem_desc_kmajor(sA, cfg.bk), desc_b0 = smem_desc_kmajor(sB, cfg.bk);
            const uint32_t desc_lo0_a = (uint32_t)desc_a0, desc_lo0_b = (uint32_t)desc_b0, desc_hi = (uint32_t)(desc_a0 >> 32);
            bool have_a = !kAres || my_tiles == 0 || mbar_wait(bar_fullA, 0, abort_flag);
            for (int64_t tile = first; tile < cfg.ntiles && have_a && !*abort_flag; tile += step, ++it) {
                // one accumulator per tile, alternating; or (two row blocks per tile) both, every tile
                const uint32_t ab = kM2 ? 0u : (it & 1);
                const uint32_t tpar = kM2 ? ((it & 1) ^ 1) : (((it >> 1) & 1) ^ 1);
                if (!mbar_wait(bar_tempty + 8 * ab, tpar, abort_flag)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + ab * kTileN;
                bool ok = true;
                int cc = 0;
                if (kTps3) {
                    // resident weights, three 64-byte k-blocks per activation stage (never with two row blocks):
                    // the taps of a kernel row in three sub-buffers, or (colshift) the taps of a kernel COLUMN
                    // reading one buffer at three row offsets
                    const uint32_t a_step = (uint32_t)cfg.a_bytes >> 4, b_step = (uint32_t)cfg.b_bytes >> 4;
                    const uint32_t t_step = cfg.colshift ? ((uint32_t)(p.W * cfg.bk) >> 4) : ((uint32_t)cfg.b_sub >> 4);
                    const uint32_t a_t = cfg.colshift ? 3 * a_step : a_step;       // between the three MMAs of a stage
                    const uint32_t a_adv = cfg.colshift ? a_step : 3 * a_step;     // from stage to stage
                    uint32_t a_lo = desc_lo0_a, b_lo = desc_lo0_b + sb * b_step;
                    const bool two = (cfg.last_ksteps == 2);
                    for (int kb = 0; kb < cfg.nkb; kb += 3) {
                        if (!mbar_wait(bar_fullB + 8 * sb, phB, abort_flag)) { ok = false; break; }
                        tc_fence_after();
                        if (issuer) {
                            mma_i8_halves(d_tmem, a_lo, b_lo, desc_hi, cfg.idesc, kb ? 1u : 0u);
                            if (two) mma_i8_halves(d_tmem, a_lo + 2, b_lo + 2, desc_hi, cfg.idesc, 1u);
                            mma_i8_halves(d_tmem, a_lo + a_t, b_lo + t_step, desc_hi, cfg.idesc, 1u);
                            if (two) mma_i8_halves(d_tmem, a_lo + a_t + 2, b_lo + t_step + 2, desc_hi, cfg.idesc, 1u);
                            mma_i8_halves(d_tmem, a_lo + 2 * a_t, b_lo + 2 * t_step, desc_hi, cfg.idesc, 1u);
                            if (two) mma_i8_halves(d_tmem, a_lo + 2 * a_t + 2, b_lo + 2 * t_step + 2, desc_hi, cfg.idesc, 1u);
                            mma_commit(bar_emptyB + 8 * sb);
                        }
                        a_lo += a_adv;
                        b_lo += b_step;
                        if (++sb == (uint32_t)cfg.nB) { sb = 0; phB ^= 1; b_lo = desc_lo0_b; }
                    }
                } else if (!kAres && cfg.bk == 128 && cfg.last_ksteps == 4) {
                    // The common deep-K form, kept as short as it gets: every k-block is four MMAs (eight
                    // with two row blocks) on a full 128-byte stage of each ring.
                    const uint32_t a_step = (uint32_t)cfg.a_bytes >> 4, b_step = (uint32_t)cfg.b_bytes >> 4;
                    uint32_t a_lo = desc_lo0_a + sa * a_step, b_lo = desc_lo0_b + sb * b_step;
                    if (kM2) {
                        if (!mbar_wait(bar_tempty + 8, tpar, abort_flag)) break;
                        tc_fence_after();
                    }
                    for (int kb = 0; kb < cfg.nkb; ++kb) {
                        if (!mbar_wait(bar_fullB + 8 * sb, phB, abort_flag) || !mbar_wait(bar_fullA + 8 * sa, phA, abort_flag)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after();
                        const uint32_t acc = kb ? 1u : 0u;
                        if (issuer) mma_i8_halves(d_tmem, a_lo, b_lo, desc_hi, cfg.idesc, acc);
                        if (issuer) mma_i8_halves(d_tmem, a_lo + 2, b_lo + 2, desc_hi, cfg.idesc, 1u);
                        if (issuer) mma_i8_halves(d_tmem, a_lo + 4, b_lo + 4, desc_hi, cfg.idesc, 1u);
                        if (issuer) mma_i8_halves(d_tmem, a_lo + 6, b_lo + 6, desc_hi, cfg.idesc, 1u);
                        if (kM2) {
                            const uint32_t a1 = a_lo + (kABytes >> 4);
                            if (issuer) mma_i8_halves(d_tmem + kTileN, a1, b_lo, desc_hi, cfg.idesc, acc);
                            if (issuer) mma_i8_halves(d_tmem + kTileN, a1 + 2, b_lo + 2, desc_hi, cfg.idesc, 1u);
                            if (issuer) mma_i8_halves(d_tmem + kTileN, a1 + 4, b_lo + 4, desc_hi, cfg.idesc, 1u);
                            if (issuer) mma_i8_halves(d_tmem + kTileN, a1 + 6, b_lo + 6, desc_hi, cfg.idesc, 1u);
                        }
                        if (issuer) mma_commit(bar_emptyA + 8 * sa);
                        if (issuer) mma_commit(bar_emptyB + 8 * sb);
                        a_lo += a_step;
                        b_lo += b_step;
                        if (++sa == (uint32_t)cfg.nA) { sa = 0; phA ^= 1; a_lo = desc_lo0_a; }
                        if (++sb == (uint32_t)cfg.nB) { sb = 0; phB ^= 1; b_lo = desc_lo0_b; }
                    }
                } else {
                    const bool uniform = (cfg.last_ksteps == (cfg.bk >> 5));      // every k-block has the same depth
                    const uint32_t a_step = (uint32_t)cfg.a_bytes >> 4, b_step = (uint32_t)cfg.b_bytes >> 4;
                    uint32_t a_lo = kAres ? desc_lo0_a : desc_lo0_a + sa * a_step;
                    uint32_t b_lo = desc_lo0_b + sb * b_step;
                    for (int kb = 0; kb < cfg.nkb; ++kb) {
                        if (!mbar_wait(bar_fullB + 8 * sb, phB, abort_flag) ||
                            (!kAres && !mbar_wait(bar_fullA + 8 * sa, phA, abort_flag))) { ok = false; break; }
                        tc_fence_after();
                        const int ksteps = (uniform || cc != cfg.cpt - 1) ? (cfg.bk >> 5) : cfg.last_ksteps;
                        if (issuer) mma_i8_halves(d_tmem, a_lo, b_lo, desc_hi, cfg.idesc, kb ? 1u : 0u);
                        for (int ks = 1; ks < ksteps; ++ks)
                            if (issuer) mma_i8_halves(d_tmem, a_lo + 2 * ks, b_lo + 2 * ks, desc_hi, cfg.idesc, 1u);
                        if (kM2) {
                            // second row block: rows 128..255 of the weight stage, second accumulator
                            if (kb == 0) {
                                if (!mbar_wait(bar_tempty + 8, tpar, abort_flag)) { ok = false; break; }
                                tc_fence_after();
                            }
                            const uint32_t a1 = a_lo + (kABytes >> 4);
                            if (issuer) mma_i8_halves(d_tmem + kTileN, a1, b_lo, desc_hi, cfg.idesc, kb ? 1u : 0u);
                            for (int ks = 1; ks < ksteps; ++ks)
                                if (issuer) mma_i8_halves(d_tmem + kTileN, a1 + 2 * ks, b_lo + 2 * ks, desc_hi, cfg.idesc, 1u);
                        }
                        if (!kAres && issuer) mma_commit(bar_emptyA + 8 * sa);
                        if (issuer) mma_commit(bar_emptyB + 8 * sb);
                        a_lo += a_step;
                        b_lo += b_step;
                        if (++sa == (uint32_t)cfg.nA) { sa = 0; phA ^= 1; if (!kAres) a_lo = desc_lo0_a; }
                        if (++sb == (uint32_t)cfg.nB) { sb = 0; phB ^= 1; b_lo = desc_lo0_b; }
                        if (!uniform && ++cc == cfg.cpt) cc = 0;
                    }
                }
                if (!ok) break;
                if (issuer) mma_commit(bar_tfull + 8 * ab);
                if (kM2 && issuer) mma_commit(bar_tfull + 8);
            }
        }
    } else if (!kPre && warp < 2 + kNumExpWarps) {
        // ---------------------------------------------------------- expanders
        const int grp = (warp - 2) >> 2;                 // which k-blocks: g % kGroups == grp
        const int et = ((warp - 2) & 3) * 32 + lane;     // 0..127 inside the group
        const int q = et & 3;                            // 32-code step inside each k-block
        const int slot0 = et >> 2;                       // rows slot0 + 32*i of the tile's sorted order
        // tile look-ahead: one tile, or kGroups tiles when every tile is a single k-block
        const int64_t look = (cfg.nkb == 1) ? kGroups : 1;
        const int64_t total = kPre ? 0 : my_tiles * cfg.nkb;   // nothing to expand in pre mode
        int64_t g = grp;                                 // this CTA's k-block counter
        int64_t tl = g / cfg.nkb;                        // local tile index of g
        int kb = (int)(g - tl * cfg.nkb);
        int cc = kb % cfg.cpt;
        uint32_t sa = (uint32_t)(g % cfg.nA), phA = (uint32_t)((g / cfg.nA) & 1);
        uint32_t sr = (uint32_t)(g % cfg.nR), phR = (uint32_t)((g / cfg.nR) & 1);
        uint32_t cur[4], nxt[4];
        auto tile_of = [&](int64_t local) -> int64_t { return local < my_tiles ? first + local * step : -1; };
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            cur[i] = kPre ? 0u : make_meta(p, tile_of(tl), slot0 + 32 * i, q);
            nxt[i] = kPre ? 0u : make_meta(p, tile_of(tl + look), slot0 + 32 * i, q);
        }
        while (g < total) {
            const int ksteps = (cc == cfg.cpt - 1) ? cfg.last_ksteps : 4;
            if (!mbar_wait_warp(bar_fullR + 8 * sr, phR, abort_flag)) break;
            if (!mbar_wait_warp(bar_emptyA + 8 * sa, phA ^ 1, abort_flag)) break;
            if (q < ksteps) {
                const uint32_t rs = sRaw + sr * cfg.raw_bytes, as = sA + sa * cfg.a_bytes;
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if ((cur[i] >> 30) != 3u) expand_task(cur[i], rs, as);
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(bar_fullA + 8 * sa);
                mbar_arrive(bar_emptyR + 8 * sr);
            }
            // advance by kGroups k-blocks
            g += kGroups;
            sa += kGroups; while (sa >= (uint32_t)cfg.nA) { sa -= cfg.nA; phA ^= 1; }
            sr += kGroups; while (sr >= (uint32_t)cfg.nR) { sr -= cfg.nR; phR ^= 1; }
            kb += kGroups;
            cc += kGroups; while (cc >= cfg.cpt) cc -= cfg.cpt;
            if (kb >= cfg.nkb) {
                int64_t adv = 0;
                while (kb >= cfg.nkb) { kb -= cfg.nkb; ++adv; }
                tl += adv;
                cc = kb % cfg.cpt;
                if (adv == look) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) cur[i] = nxt[i];
                } else {
#pragma unroll
                    for (int i = 0; i < 4; ++i) cur[i] = make_meta(p, tile_of(tl), slot0 + 32 * i, q);
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) nxt[i] = make_meta(p, tile_of(tl + look), slot0 + 32 * i, q);
            }
        }
    } else {
        // ---------------------------------------------------------- epilogue
        // Warp w may read tensor-memory lanes 32*(w%4)..+31.  The warps that share a quarter (one, or
        // three in pre mode) take alternate 32-pixel chunks; with duplicated rows the two quarters
        // holding the same rows share the chunks as well.
        const int quarter = warp & 3;
        const int first_epi = kThreads / 32 - cfg.epi_warps;               // epilogue warps are the last epi_warps warps
        const int ew = warp - first_epi;                                   // 0 .. epi_warps-1
        // how many epilogue warps share a quarter, and this warp's rank among them
        auto count_q = [&](int q) { const int f = first_epi + ((q - first_epi) & 3); return (kThreads / 32 - 1 - f) / 4 + 1; };
        const int my_rank = (warp - (first_epi + ((quarter - first_epi) & 3))) >> 2;
        const int row0 = cfg.dup ? (quarter & 1) * 32 : quarter * 32;       // first row (within the block) of this warp
        const int cstride = cfg.dup ? count_q(quarter & 1) + count_q((quarter & 1) + 2) : count_q(quarter);
        const int cfirst = (cfg.dup && (quarter >> 1)) ? count_q(quarter & 1) + my_rank : my_rank;
        const uint32_t my_stage = sOut + (uint32_t)ew * (cfg.out_bufs * kWarpStage);
        uint32_t it = 0, stg_count = 0;
        bool alive = true;
        int scale_blk = -1, shift = 0;
        float scale = 0.f;
        const ActFast rq_fast = act_fast_setup(kRQ ? p.rq_alpha : 1.0f, kRQ ? p.rq_kind : 0);
        for (int64_t tile = first; tile < cfg.ntiles && alive; tile += step, ++it) {
          // a tile is one row block (accumulators alternate between tiles), or two (one accumulator each)
          for (int half = 0; half <= kM2; ++half) {
            const uint32_t ab = kM2 ? (uint32_t)half : (it & 1);
            const uint32_t tpar = kM2 ? (it & 1) : ((it >> 1) & 1);
            // tile indices fit 32 bits (checked on the host): 32-bit divisions, a fraction of the 64-bit ones' cost,
            // which every epilogue warp would otherwise pay in front of each tile
            const uint32_t nt = (uint32_t)tile / (uint32_t)cfg.nbt;
            const int blk = ((int)((uint32_t)tile - nt * (uint32_t)cfg.nbt) << kM2) + half;
            int64_t n0;
            if (cfg.tiles_per_image) {
                const uint32_t img = nt / (uint32_t)cfg.tiles_per_image, tin = nt - img * (uint32_t)cfg.tiles_per_image;
                n0 = ((int64_t)img * p.Ho + (int64_t)tin * cfg.th) * (int64_t)p.Wo;
            } else {
                n0 = (int64_t)nt * cfg.npix;
            }
            const int nvalid = (int)min((int64_t)cfg.npix, p.N - n0);
            const int m = blk * kBlockRows + row0 + lane;
            const bool row_ok = m < p.M;
            if (blk != scale_blk) {
                // the row's scale: loaded when the row block changes (never again for layers of one row block)
                scale_blk = blk;
                scale = 0.f;
                shift = 0;
                if (row_ok) {
                    scale = __fmul_rn(__ldg(p.wstep + m), p.act_step);
                    shift = (!kPre && __ldg(p.kind + m) == kFixed4) ? 4 : 0;   // expanders store Fixed-4 codes as 16 * value
                }
            }
            if (!mbar_wait_warp(bar_tfull + 8 * ab, tpar, abort_flag)) { alive = false; break; }
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + ab * kTileN;
            const int nchunks = (nvalid + 31) >> 5;
            auto release_tmem = [&]() {
                // all accumulators of this tile are in registers: hand the buffer back
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_tempty + 8 * ab);
            };
            if (blk * kBlockRows + row0 >= p.M || cfirst >= nchunks) {      // no valid row, or no chunk, for this warp
                release_tmem();
                continue;
            }
            // Output one 32-pixel chunk held in registers.
            auto emit = [&](const uint32_t (&v)[32], int c) {
                const int jmax = min(32, nvalid - c * 32);
                if (kRQ) {
                    // y as in the fp32 epilogue, then the activation quantizer's arithmetic on it;
                    // one code byte per output, 32 pixels x 32 rows = 1 KB per chunk
                    if (use_tma_store) {
                        const bool tail = cfg.tail_rows && (c == (cfg.npix >> 5));
                        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                        __syncwarp();
                        // pass 1, branch-free so that the 32 dependent chains interleave: the division-free
                        // code of every value, and one bit per value whose code the division must decide
                        // (scaled value u = acc * g with g = scale / alpha * Q folded into one factor: a few
                        // ulps from the defining chain of roundings, far inside the 1e-4 guard band)
                        uint32_t undecided = rq_fast.ok ? 0u : 0xffffffffu;
                        const float g = __fmul_rn(__fmul_rn(scale, rq_fast.r), rq_fast.q);
                        const float u_lo = __fmul_rn(rq_fast.lo, rq_fast.q), u_hi = rq_fast.q;
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const float kMagic = 12582912.0f;
                            float u = __fmul_rn(__int2float_rn((int)v[j] >> shift), g);
                            u = fminf(fmaxf(u, u_lo), u_hi);
                            const float sgm = __fadd_rn(u, kMagic);
                            const float dev = __fsub_rn(u, __fsub_rn(sgm, kMagic));
                            undecided |= (fabsf(dev) <= 0.4999f ? 0u : 1u) << j;
                            asm volatile("st.shared.u8 [%0], %1;" ::"r"(my_stage + j * 32 + lane), "r"(__float_as_uint(sgm)) : "memory");
                        }
                        // pass 2, rare: those values again by the definition
                        while (undecided) {
                            const int j = __ffs(undecided) - 1;
                            undecided &= undecided - 1;
                            uint32_t a = 0;
#pragma unroll
                            for (int jj = 0; jj < 32; ++jj) a = (jj == j) ? v[jj] : a;     // registers cannot be indexed
                            const float y = __fmul_rn(__int2float_rn((int)a >> shift), scale);
                            const uint32_t code = (uint32_t)act_code(y, p.rq_alpha, p.rq_kind);
                            asm volatile("st.shared.u8 [%0], %1;" ::"r"(my_stage + j * 32 + lane), "r"(code) : "memory");
                        }
                        fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0)
                            tma_store_2d(tail ? &maps.rq_tail : &maps.rq_full, my_stage, blk * kBlockRows + row0, (int)(n0 + c * 32));
                    } else if (row_ok) {
                        int8_t* o = p.rq_codes + (n0 + c * 32) * p.ld_codes + m;
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            if (j < jmax) {
                                const float y = __fmul_rn(__int2float_rn((int)v[j] >> shift), scale);
                                o[(int64_t)j * p.ld_codes] = (int8_t)act_code_exact(y, p.rq_alpha, p.rq_kind, rq_fast);
                            }
                        }
                    }
                } else if (use_tma_store) {
                    const bool tail = cfg.tail_rows && (c == (cfg.npix >> 5));
                    const int nsub = acc_out ? 2 : 1;
                    for (int sub = 0; sub < nsub; ++sub) {
                        const uint32_t stg = my_stage + (cfg.out_bufs == 2 ? (stg_count & 1) * kWarpStage : 0);
                        ++stg_count;
                        if (lane == 0) {
                            if (cfg.out_bufs == 2) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                            else asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                        }
                        __syncwarp();                    // the buffer's previous store has been read out
                        if (!out_mn) {
                            // [pixel][row]: the warp writes 128 contiguous bytes per pixel
                            const uint32_t a0 = stg + lane * 4;
#pragma unroll
                            for (int j = 0; j < 32; ++j) {
                                const int a = (int)v[j] >> shift;
                                const uint32_t w = sub ? (uint32_t)a : __float_as_uint(__fmul_rn(__int2float_rn(a), scale));
                                asm volatile("st.shared.b32 [%0], %1;" ::"r"(a0 + j * 128), "r"(w) : "memory");
                            }
                        } else {
                            // [row][pixel], 16-byte chunks swizzled by row (matches the 128-byte-swizzled store map)
                            const uint32_t a0 = stg + lane * 128;
#pragma unroll
                            for (int cch = 0; cch < 8; ++cch) {
                                uint32_t w[4];
#pragma unroll
                                for (int t = 0; t < 4; ++t) {
                                    const int a = (int)v[4 * cch + t] >> shift;
                                    w[t] = sub ? (uint32_t)a : __float_as_uint(__fmul_rn(__int2float_rn(a), scale));
                                }
                                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                                             ::"r"(a0 + ((cch ^ (lane & 7)) << 4)), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
                            }
                        }
                        fence_proxy_async_smem();
                        __syncwarp();                    // chunk complete in shared memory
                        if (lane == 0) {
                            const CUtensorMap* map = sub ? (tail ? &maps.acc_tail : &maps.acc_full)
                                                         : (tail ? &maps.out_tail : &maps.out_full);
                            const int cm = blk * kBlockRows + row0, cn = (int)(n0 + c * 32);
                            if (!out_mn) tma_store_2d(map, stg, cm, cn); else tma_store_2d(map, stg, cn, cm);
                        }
                    }
                } else if (row_ok) {
                    // direct stores: outputs whose leading dimension or base rules out bulk stores
                    if (!out_mn) {
                        float* o = p.out + (n0 + c * 32) * p.ld_out + m;
                        int32_t* oa = acc_out ? acc_out + (n0 + c * 32) * p.ld_out + m : nullptr;
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            if (j < jmax) {
                                const int a = (int)v[j] >> shift;
                                o[(int64_t)j * p.ld_out] = __fmul_rn(__int2float_rn(a), scale);
                                if (oa) oa[(int64_t)j * p.ld_out] = a;
                            }
                        }
                    } else {
                        float* o = p.out + (int64_t)m * p.ld_out + n0 + c * 32;
                        int32_t* oa = acc_out ? acc_out + (int64_t)m * p.ld_out + n0 + c * 32 : nullptr;
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
            };
            // two register sets: the load of this warp's next chunk is in flight while the current one is emitted
            uint32_t va[32], vb[32];
            tmem_ld_issue(taddr + cfirst * 32, va);
            tmem_ld_wait(va);
            for (int c = cfirst; c < nchunks; c += 2 * cstride) {
                const int c1 = c + cstride, c2 = c + 2 * cstride;
                const bool more1 = c1 < nchunks;
                if (more1) tmem_ld_issue(taddr + c1 * 32, vb); else release_tmem();
                emit(va, c);
                if (more1) {
                    tmem_ld_wait(vb);
                    const bool more2 = c2 < nchunks;
                    if (more2) tmem_ld_issue(taddr + c2 * 32, va); else release_tmem();
                    emit(vb, c1);
                    if (more2) tmem_ld_wait(va);
                }
            }
          }
        }
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    }

    // ---------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
    }
    if (threadIdx.x == 0 && s_abort) atomicMax(p.status, (uint32_t)RMSMP_ERR_TIMEOUT);
}

// ------------------------------------------------------------------ host side

EncodeTiledFn encode_fn() { return tensor_map_encoder(); }

// Tensor maps of the activation codes for boxes of `bk` channels x th output rows x tb images
// (see act_parity_split: one map, or one per parity sub-grid of a stride-2 layer).
bool encode_act_maps(EncodeTiledFn enc, const Problem& p, int bk, int th, int tb, CUtensorMapSwizzle swz, CUtensorMap out[4])
{
    const cuuint64_t pitch = (cuuint64_t)p.pix_pitch;
    if (act_parity_split(p)) {
        for (int py = 0; py < 2; ++py)
            for (int px = 0; px < 2; ++px) {
                const cuuint64_t gdim[4] = {(cuuint64_t)p.Cin, (cuuint64_t)((p.W - px + 1) / 2), (cuuint64_t)((p.H - py + 1) / 2), (cuuint64_t)p.B};
                const cuuint64_t gstr[3] = {2 * pitch, 2 * pitch * p.W, pitch * p.W * p.H};
                const cuuint32_t box[4] = {(cuuint32_t)bk, (cuuint32_t)p.Wo, (cuuint32_t)th, (cuuint32_t)tb};
                const cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
                const int8_t* base = p.act + ((int64_t)py * p.W + px) * p.pix_pitch;
                if (enc(&out[py * 2 + px], CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<int8_t*>(base), gdim, gstr, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
                    return false;
            }
        return true;
    }
    const cuuint64_t gdim[4] = {(cuuint64_t)p.Cin, (cuuint64_t)p.W, (cuuint64_t)p.H, (cuuint64_t)p.B};
    const cuuint64_t gstr[3] = {pitch, pitch * p.W, pitch * p.W * p.H};
    const cuuint32_t box[4] = {(cuuint32_t)bk, (cuuint32_t)(p.Wo * p.stride), (cuuint32_t)(th * p.stride), (cuuint32_t)tb};
    const cuuint32_t estr[4] = {1u, (cuuint32_t)p.stride, (cuuint32_t)p.stride, 1u};
    return enc(&out[0], CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<int8_t*>(p.act), gdim, gstr, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool plan(const Problem& p, TensorCfg& c)
{
    if (p.pix_pitch % 16 != 0 || p.Cin % 16 != 0) return false;
    if ((reinterpret_cast<uintptr_t>(p.act) & 15) != 0) return false;
    if (!p.wexp && p.raw_stage_bytes <= 0) return false;
    if (p.wexp && (reinterpret_cast<uintptr_t>(p.wexp) & 15) != 0) return false;
    const int64_t hw = (int64_t)p.Ho * p.Wo;
    if (p.Wo > kTileN || (int64_t)p.Wo * p.stride > 256) return false;
    if (hw <= kTileN) {
        c.th = p.Ho;
        c.tb = (int)std::min<int64_t>(kTileN / hw, p.B);
        c.tiles_per_image = 0;
        c.ntiles_n = (p.B + c.tb - 1) / c.tb;
    } else {
        int th = 1;
        for (int d = 1; d <= p.Ho; ++d)
            if (p.Ho % d == 0 && (int64_t)d * p.Wo <= kTileN) th = d;
        c.th = th; c.tb = 1;
        c.tiles_per_image = p.Ho / th;
        c.ntiles_n = (int64_t)p.B * c.tiles_per_image;
    }
    if ((int64_t)c.th * p.stride > 256) return false;
    c.npix = c.tb * c.th * p.Wo;
    c.n_mma = (c.npix + 15) / 16 * 16;
    c.ntiles = c.ntiles_n * p.nblocks;
    if (c.ntiles >= (1ll << 31)) return false;
    c.m2 = 0;
    c.nbt = p.nblocks;
    c.tps = 1;
    c.b_sub = 0;
    c.colshift = 0;
    c.pre = p.wexp ? 1 : 0;
    c.fill = 0;
    if (!p.wexp && p.nblocks == 1 && !p.rq_codes) {
        // no workspace, but the whole row block's expanded weights would stay resident: the CTA expands them once
        // itself and the layer runs in the workspace form
        const int bk = ((p.Cin % 128 != 0) && (p.Cin % 128 <= 64)) ? 64 : 128;
        const int64_t nkb = (int64_t)p.kh * p.kw * ((p.Cin + bk - 1) / bk);
        if (nkb * kBlockRows * bk <= 72 * 1024) { c.pre = 1; c.fill = 1; }
    }
    // 64-byte k-blocks when a 128-byte row would be at most half used by the (last) channel chunk
    c.bk = (c.pre && (p.Cin % 128 != 0) && (p.Cin % 128 <= 64)) ? 64 : 128;
    c.a_bytes = kBlockRows * c.bk;
    c.b_bytes = kTileN * c.bk;
    c.cpt = (p.Cin + c.bk - 1) / c.bk;
    c.nkb = p.kh * p.kw * c.cpt;
    c.last_ksteps = (p.Cin - (c.cpt - 1) * c.bk + 31) / 32;
    c.tx_bytes = (uint32_t)c.npix * (uint32_t)c.bk;
    // kind::i8: int32 accumulate (bits 4-5 = 2), signed 8-bit A and B (bits 7-9, 10-12 = 1),
    // both K-major, N/8 at bit 17, M/16 at bit 24
    c.idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(c.n_mma >> 3) << 17) | ((uint32_t)(kBlockRows >> 4) << 24);
    c.tail_rows = c.npix & 31;
    c.tma_store = 0;
    c.dup = 0;
    c.ares = 0;
    c.epi_warps = kNumEpiWarps;
    if (c.pre) {
        c.nA = (c.bk == 64) ? 6 : 3; c.nB = (c.bk == 64) ? 8 : 4; c.nR = 0; c.raw_bytes = 0; c.out_bufs = 1;
        c.epi_warps = kNumExpWarps + kNumEpiWarps - 1;   // warp 2 fetches the weights (unless they are resident)
        c.dup = (p.M <= 64) ? 1 : 0;
        if (p.nblocks == 1 && (int64_t)c.nkb * c.a_bytes <= 72 * 1024) {
            c.ares = 1;
            c.epi_warps = kNumExpWarps + kNumEpiWarps;
            c.nA = c.nkb;
            const int64_t left = kSmemLimit - (1024 + 64 * kMaxRing) - (int64_t)c.nkb * c.a_bytes -
                                 (int64_t)c.epi_warps * kWarpStage;
            c.nB = (int)std::min<int64_t>(kMaxRing, left / c.b_bytes);
        }
        c.tps = 1;
        c.b_sub = c.b_bytes;
        if (c.ares && c.bk == 64 && c.cpt == 1 && p.kw == 3 && c.last_ksteps <= 2) {
            c.tps = 3;
            c.b_sub = (c.n_mma * c.bk + 1023) / 1024 * 1024;
            c.b_bytes = c.tps * c.b_sub;
            if (p.kh == 3 && p.stride == 1 && p.Wo == p.W && c.tb == 1 && p.W % 8 == 0 && c.npix == c.th * p.W) {
                c.colshift = 1;
                c.tx_bytes = (uint32_t)((c.th + 2) * p.W * c.bk);
                c.b_bytes = ((c.th + 2) * p.W * c.bk + 1023) / 1024 * 1024;
            }
            const int64_t left = kSmemLimit - (1024 + 64 * kMaxRing) - (int64_t)c.nkb * c.a_bytes -
                                 (int64_t)c.epi_warps * kWarpStage;
            c.nB = (int)std::min<int64_t>(kMaxRing, left / c.b_bytes);
            if (c.nB < 2) { c.tps = 1; c.colshift = 0; c.tx_bytes = (uint32_t)c.npix * (uint32_t)c.bk; c.b_bytes = kTileN * c.bk; c.b_sub = c.b_bytes; c.nB = (int)std::min<int64_t>(kMaxRing, left / c.b_bytes); }
        }
        // Two row blocks per tile pay when K is long (the two accumulators' epilogue is only half
        // hidden behind the next tile's MMAs) and when the halved tile count does not cost more in
        // idle SMs of the last wave than the ~20 % a double tile saves.
        const int64_t sms = sm_count();
        const int64_t waves1 = (c.ntiles + sms - 1) / sms, waves2 = (c.ntiles / 2 + sms - 1) / sms;
        if (!c.ares && !c.dup && c.bk == 128 && p.nblocks % 2 == 0 && c.nkb >= 16 && 16 * waves2 < 10 * waves1) {
            c.m2 = 1;
            c.nbt = p.nblocks / 2;
            c.ntiles = c.ntiles_n * c.nbt;
            c.a_bytes = 2 * kABytes;
            c.nA = 2; c.nB = 3;
        }
        c.smem_bytes = (uint32_t)(c.nA * c.a_bytes + c.nB * c.b_bytes + c.epi_warps * c.out_bufs * kWarpStage + 1024 +
                                  64 * kMaxRing);
        return true;
    }
    // shared-memory budget: rings as deep as fit
    c.raw_bytes = ((uint32_t)p.raw_stage_bytes + 1023u) & ~1023u;
    const int fixed = 1024 /*alignment*/ + 64 * kMaxRing /*barriers*/;
    struct Choice { int nA, nB, nR, ob; };
    const Choice order[] = {{3, 4, 3, 2}, {3, 4, 3, 1}, {3, 3, 3, 2}, {2, 3, 3, 2}, {2, 3, 2, 1}, {2, 2, 2, 1}};
    for (const Choice& ch : order) {
        const int64_t need = (int64_t)ch.nA * kABytes + (int64_t)ch.nB * kBBytes + (int64_t)ch.nR * c.raw_bytes +
                             (int64_t)kNumEpiWarps * ch.ob * kWarpStage + fixed;
        if (need <= kSmemLimit) {
            c.nA = ch.nA; c.nB = ch.nB; c.nR = ch.nR; c.out_bufs = ch.ob; c.smem_bytes = (uint32_t)need;
            return true;
        }
    }
    return false;
}

}  // namespace

EncodeTiledFn tensor_map_encoder()
{
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
        else
            cudaGetLastError();
    }
    return fn;
}

bool encode_act_maps_4(const Problem& p, int bk, int th, int tb, void* maps4)
{
    EncodeTiledFn enc = encode_fn();
    return enc && encode_act_maps(enc, p, bk, th, tb, bk == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                                  static_cast<CUtensorMap*>(maps4));
}

bool tensor_supported(const Problem& p)
{
    TensorCfg c;
    return plan(p, c) && encode_fn() != nullptr;
}

rmsmp_status launch_tensor(const Problem& p, cudaStream_t st)
{
    if (pair_supported(p)) return launch_pair(p, st);
    TensorCfg c;
    if (!plan(p, c)) return RMSMP_ERR_VARIANT;
    EncodeTiledFn enc = encode_fn();
    if (!enc) return RMSMP_ERR_CUDA;
    Maps mp;
    memset(&mp, 0, sizeof(mp));
    if (!encode_act_maps(enc, p, c.bk, c.colshift ? c.th + 2 : c.th, c.tb, c.bk == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B, mp.act))
        return RMSMP_ERR_CUDA;
    // packed weight regions: rows of Kp/2 (4-bit) and Kp (8-bit) bytes, boxes of 16 rows x one k-block
    auto make_w = [&](CUtensorMap* m, const uint8_t* base, int rows, int pitch, int box_bytes) -> bool {
        if (rows <= 0) return true;
        const cuuint64_t gd[2] = {(cuuint64_t)pitch, (cuuint64_t)rows};
        const cuuint64_t gs[1] = {(cuuint64_t)pitch};
        const cuuint32_t bx[2] = {(cuuint32_t)box_bytes, (cuuint32_t)kRawBoxRows};
        const cuuint32_t es[2] = {1, 1};
        return enc(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(base), gd, gs, bx, es,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    };
    if (!make_w(&mp.q4, p.q4, p.nP + p.nF4, p.Kp / 2, 64) || !make_w(&mp.q8, p.q8, p.n8, p.Kp, 128))
        return RMSMP_ERR_CUDA;
    if (p.wexp) {
        const cuuint64_t gd[2] = {(cuuint64_t)p.Kp, (cuuint64_t)p.M};
        const cuuint64_t gs[1] = {(cuuint64_t)p.Kp};
        const cuuint32_t bx[2] = {(cuuint32_t)c.bk, (cuuint32_t)(c.dup ? kBlockRows / 2 : (c.m2 ? 2 * kBlockRows : kBlockRows))};
        const cuuint32_t es[2] = {1, 1};
        if (enc(&mp.wexp, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t*>(p.wexp), gd, gs, bx, es,
                CU_TENSOR_MAP_INTERLEAVE_NONE, c.bk == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return RMSMP_ERR_CUDA;
    }

    const bool ld_ok = !p.rq_codes && (p.ld_out % 4 == 0) && (p.out_mn ? p.N % 4 == 0 : p.M % 4 == 0) && ((reinterpret_cast<uintptr_t>(p.out) & 15) == 0) &&
                       (!p.acc || (reinterpret_cast<uintptr_t>(p.acc) & 15) == 0);
    if (p.rq_codes) {
        // re-quantized output: [N][ld_codes] code bytes, boxes of 32 rows (bytes) x 32 pixels
        if (!c.pre || p.out_mn) return RMSMP_ERR_VARIANT;
        // bulk stores clip at 16-byte granules of the innermost dimension: a row count that is not a
        // multiple of 16 bytes would spill into the padding columns, so such outputs take direct stores
        if (p.M % 16 == 0 && p.ld_codes % 16 == 0 && (reinterpret_cast<uintptr_t>(p.rq_codes) & 15) == 0) {
            auto make = [&](CUtensorMap* m, int rows) -> bool {
                const cuuint32_t es[2] = {1, 1};
                const cuuint64_t gs[1] = {(cuuint64_t)p.ld_codes};
                const cuuint64_t gd[2] = {(cuuint64_t)p.M, (cuuint64_t)p.N};
                const cuuint32_t bx[2] = {32u, (cuuint32_t)rows};
                return enc(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, p.rq_codes, gd, gs, bx, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
            };
            bool ok = make(&mp.rq_full, 32);
            if (ok && c.tail_rows) ok = make(&mp.rq_tail, c.tail_rows);
            c.tma_store = ok ? 1 : 0;
        }
    }
    if (ld_ok && (!p.out_mn || c.tail_rows == 0)) {
        auto make = [&](CUtensorMap* m, void* base, CUtensorMapDataType dt, int rows) -> bool {
            const cuuint32_t es[2] = {1, 1};
            const cuuint64_t gs[1] = {(cuuint64_t)p.ld_out * 4};
            if (!p.out_mn) {
                const cuuint64_t gd[2] = {(cuuint64_t)p.M, (cuuint64_t)p.N};
                const cuuint32_t bx[2] = {32u, (cuuint32_t)rows};
                return enc(m, dt, 2, base, gd, gs, bx, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                           CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
            }
            const cuuint64_t gd[2] = {(cuuint64_t)p.N, (cuuint64_t)p.M};
            const cuuint32_t bx[2] = {32u, 32u};
            return enc(m, dt, 2, base, gd, gs, bx, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                       CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
        };
        bool ok = make(&mp.out_full, p.out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 32);
        if (ok && c.tail_rows) ok = make(&mp.out_tail, p.out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, c.tail_rows);
        if (ok && p.acc) ok = make(&mp.acc_full, p.acc, CU_TENSOR_MAP_DATA_TYPE_INT32, 32);
        if (ok && p.acc && c.tail_rows) ok = make(&mp.acc_tail, p.acc, CU_TENSOR_MAP_DATA_TYPE_INT32, c.tail_rows);
        c.tma_store = ok ? 1 : 0;
    }

    // the kernel's form (see tensor_kernel): [mode][two row blocks][1: re-quantizing epilogue, 2: plain fp32 [N][M] bulk-store output]
    typedef void (*KernelFn)(const Problem, const TensorCfg, const Maps);
    static const KernelFn table[4][2][3] = {
        {{tensor_kernel<0, 0, 0, 0>, nullptr, tensor_kernel<0, 0, 0, 1>}, {nullptr, nullptr, nullptr}},
        {{tensor_kernel<0, 0, 1, 0>, tensor_kernel<0, 1, 1, 0>, tensor_kernel<0, 0, 1, 1>},
         {tensor_kernel<1, 0, 1, 0>, tensor_kernel<1, 1, 1, 0>, tensor_kernel<1, 0, 1, 1>}},
        {{tensor_kernel<0, 0, 2, 0>, tensor_kernel<0, 1, 2, 0>, tensor_kernel<0, 0, 2, 1>}, {nullptr, nullptr, nullptr}},
        {{tensor_kernel<0, 0, 3, 0>, tensor_kernel<0, 1, 3, 0>, tensor_kernel<0, 0, 3, 1>}, {nullptr, nullptr, nullptr}},
    };
    const int mode = !c.pre ? 0 : (!c.ares ? 1 : (c.tps > 1 ? 3 : 2));
    const int i2 = c.m2 ? 1 : 0;
    const int io = p.rq_codes ? 1 : ((c.tma_store && !p.out_mn && !p.acc) ? 2 : 0);
    const KernelFn fn = table[mode][i2][io];
    if (!fn) return RMSMP_ERR_VARIANT;
    static bool attr_set[4][2][3][kMaxDevices] = {};
    if (!ensure_smem_attr(reinterpret_cast<const void*>(fn), kSmemLimit, attr_set[mode][i2][io])) return RMSMP_ERR_CUDA;
    const int grid = (int)std::min<int64_t>(c.ntiles, sm_count());
    fn<<<grid, kThreads, c.smem_bytes, st>>>(p, c, mp);
    if (cudaGetLastError() != cudaSuccess) return RMSMP_ERR_CUDA;
    return RMSMP_OK;
}

}  // namespace rmsmp
