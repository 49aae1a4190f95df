// Tensor-core variant of the contraction for sm_100a.
//
// One persistent CTA per SM walks over output tiles of 128 weight rows x up to 256 pixels.
// Warp roles:
//   warp 0      TMA producer: activation-code tiles (the B operand) global -> shared memory,
//               128-byte swizzled, one 4-D box per k-block; for a convolution the box is the
//               window of input pixels one filter tap needs (zero fill outside the image = the
//               padding), so no im2col buffer exists anywhere.
//   warp 1      allocates tensor memory, issues tcgen05.mma (kind::i8, int32 accumulators in
//               tensor memory, two 256-column buffers so tile i+1 is computed while tile i
//               is being written out).
//   warps 2-9   expanders: fetch the packed 4-bit / 8-bit weight codes of the tile's rows,
//               expand them to int8 in registers and store them into shared memory in the
//               K-major 128-byte-swizzled layout the MMA reads (the A operand).  Rows are
//               fetched group by group (PoT, Fixed-4, Fixed-8) but written to the row position
//               of their ORIGINAL index, so accumulator lanes are in original row order and
//               the output needs no scatter.
//   warps 10+   epilogue: tcgen05.ld the accumulators, undo the x16 of Fixed-4 rows, convert,
//               scale by wstep*act_step, store.
// Every wait on an mbarrier is bounded; when one runs out the kernel records
// RMSMP_ERR_TIMEOUT in the packed buffer's status word, all roles leave their loops, tensor
// memory is freed and the kernel returns.
#include <cuda.h>
#include <cstring>
#include "common.cuh"
#include "decode.cuh"

namespace rmsmp {

namespace {

constexpr int kStages = 4;
constexpr int kTileN = 256;                      // pixels per tile (max) = TMEM columns per buffer
constexpr int kABytes = kBlockRows * 128;        // 16 KB: 128 rows x 128 B (one k-block)
constexpr int kBBytes = kTileN * 128;            // 32 KB
constexpr int kNumExpWarps = 8;
constexpr int kNumEpiWarps = 4;                 // kEpiPerQuarter warps share a tensor-memory quarter, alternating 32-pixel chunks
constexpr int kEpiPerQuarter = kNumEpiWarps / 4;
constexpr int kThreads = 32 * (2 + kNumExpWarps + kNumEpiWarps);
constexpr int kWarpStage = 32 * 32 * 4;          // 4 KB: 32 pixels x 32 rows of fp32/int32, one epilogue warp's chunk
constexpr int kStageOut = kNumEpiWarps * kWarpStage;   // one private buffer per epilogue warp
constexpr int kSmemBytes = kStages * (kABytes + kBBytes) + kStageOut + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr long long kWaitCycles = 2000000000LL;  // ~1 s: far beyond any legitimate wait

struct TensorCfg {
    int tb, th;            // images / output rows per tile
    int npix;              // pixels per full tile = tb*th*Wo
    int n_mma;             // npix rounded up to 16
    int tiles_per_image;   // Ho/th when tb == 1 and th < Ho, else 0
    int64_t ntiles_n;
    int64_t ntiles;        // ntiles_n * nblocks
    int cpt;               // 128-channel chunks per tap
    int nkb;               // k-blocks per tile = taps * cpt
    uint32_t idesc;
    uint32_t tx_bytes;     // bytes one activation box brings
    int tma_store;         // 1: output chunks leave through shared memory and bulk tensor stores
    int tail_rows;         // npix % 32: height of the last chunk of a tile (0: none)
};

struct StoreMaps {         // bulk-store tensor maps: fp32 output and int32 accumulators, full and tail chunk
    CUtensorMap out_full, out_tail, acc_full, acc_tail;
};

// ------------------------------------------------------------------ PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void* p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false if it gave up (or another role already did).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > kWaitCycles) { *abort_flag = 1; return false; }
    }
}
// Whole-warp form: lane 0 polls, the verdict is made uniform, and the warp-level vote orders the
// other lanes' later accesses after lane 0's observation of the barrier.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag)
{
    bool ok = true;
    if ((threadIdx.x & 31) == 0) ok = mbar_wait(bar, parity, abort_flag);
    return __all_sync(0xffffffffu, ok);
}
__device__ __forceinline__ void fence_proxy_async_smem()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0,
                                            int c1, int c2, int c3)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}

__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int c0, int c1)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(map), "r"(src), "r"(c0), "r"(c1) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}

// Shared-memory matrix descriptor: K-major, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFFu);
    d |= (uint64_t)1 << 16;              // leading byte offset (unused with swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;    // stride byte offset
    d |= (uint64_t)1 << 46;              // descriptor version of this architecture
    d |= (uint64_t)2 << 61;              // 128-byte swizzle
    return d;
}
__device__ __forceinline__ void mma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                       uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
                 : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t v[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// ------------------------------------------------------------------ expander state

// What an expander thread needs to know about one of its two rows in a tile.
struct RowTask {
    const uint8_t* src;   // start of the packed row (4-bit or 8-bit region)
    int meta;             // bits 0-7: destination row in the tile, bits 8-9: kind, 3 = no row
};

__device__ __forceinline__ RowTask make_task(const Problem& p, int64_t tile, int slot_in_tile)
{
    RowTask t;
    t.src = p.q4;
    t.meta = 3 << 8;
    if (tile < 0) return t;
    const int blk = (int)(tile % p.nblocks);
    const int4 b0 = __ldg(reinterpret_cast<const int4*>(p.blocks + 8 * blk));
    const int2 b1 = __ldg(reinterpret_cast<const int2*>(p.blocks + 8 * blk + 4));
    const int nP = b0.y, nF = b0.w, nE = b1.y;
    int kind, packed;
    if (slot_in_tile < nP) { kind = kPoT4; packed = b0.x + slot_in_tile; }
    else if (slot_in_tile < nP + nF) { kind = kFixed4; packed = p.nP + b0.z + (slot_in_tile - nP); }
    else if (slot_in_tile < nP + nF + nE) { kind = kFixed8; packed = p.nP + p.nF4 + b1.x + (slot_in_tile - nP - nF); }
    else return t;
    const int row = __ldg(p.perm + packed) - blk * kBlockRows;
    t.src = (kind == kFixed8) ? p.q8 + (size_t)(packed - p.nP - p.nF4) * p.Kp
                              : p.q4 + (size_t)packed * (p.Kp >> 1);
    t.meta = row | (kind << 8);
    return t;
}

struct RawBuf {
    uint4 lo[2], hi[2];   // per task: 16 bytes (4-bit rows) or 32 bytes (8-bit rows)
    int meta[2];
};

__device__ __forceinline__ void exp_load(RawBuf& r, const RowTask task[2], int koff, bool active)
{
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        r.meta[j] = active ? task[j].meta : (3 << 8);
        const int kind = (r.meta[j] >> 8) & 3;
        if (kind == kFixed8) {
            const uint4* s = reinterpret_cast<const uint4*>(task[j].src + koff);
            r.lo[j] = __ldg(s);
            r.hi[j] = __ldg(s + 1);
        } else if (kind != 3) {
            r.lo[j] = __ldg(reinterpret_cast<const uint4*>(task[j].src + (koff >> 1)));
        }
    }
}

__device__ __forceinline__ void exp_store(const RawBuf& r, uint32_t a_stage, int q)
{
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        const int kind = (r.meta[j] >> 8) & 3;
        if (kind == 3) continue;
        const int row = r.meta[j] & 0xFF;
        uint32_t w[8];
        if (kind == kFixed8) {
            w[0] = r.lo[j].x; w[1] = r.lo[j].y; w[2] = r.lo[j].z; w[3] = r.lo[j].w;
            w[4] = r.hi[j].x; w[5] = r.hi[j].y; w[6] = r.hi[j].z; w[7] = r.hi[j].w;
        } else if (kind == kPoT4) {
            expand_pot_chunk(r.lo[j], w);
        } else {
            expand_fixed4_chunk_x16(r.lo[j], w);
        }
        const uint32_t base = a_stage + row * 128;
        const uint32_t sw = row & 7;
        const uint32_t a0 = base + (((2 * q) ^ sw) << 4), a1 = base + (((2 * q + 1) ^ sw) << 4);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a0), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a1), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7]) : "memory");
    }
}

// ------------------------------------------------------------------ the kernel

__global__ void __launch_bounds__(kThreads, 1)
tensor_kernel(const Problem p, const TensorCfg cfg, const __grid_constant__ CUtensorMap act_map,
              const __grid_constant__ StoreMaps smaps)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sA = smem_base;
    const uint32_t sB = smem_base + kStages * kABytes;
    const uint32_t sOut = sB + kStages * kBBytes;
    const uint32_t sBar = sOut + kStageOut;
    // barriers: full[kStages], empty[kStages], tmem_full[2], tmem_empty[2]
    const uint32_t bar_full = sBar, bar_empty = sBar + 8 * kStages;
    const uint32_t bar_tfull = sBar + 16 * kStages, bar_tempty = bar_tfull + 16;
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(bar_full + 8 * s, 1 + kNumExpWarps);   // TMA producer + one arrival per expander warp
            mbar_init(bar_empty + 8 * s, 1);                  // tcgen05.commit
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_tfull + 8 * b, 1);                  // tcgen05.commit
            mbar_init(bar_tempty + 8 * b, kNumEpiWarps);      // one arrival per epilogue warp
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
    const int taps_w = p.kw;

    if (warp == 0) {
        // ---------------------------------------------------------- TMA producer
        if (lane == 0) {
            uint32_t g = 0;
            for (int64_t tile = first; tile < cfg.ntiles && !*abort_flag; tile += step) {
                const int64_t nt = tile / p.nblocks;
                int b0, h0;
                if (cfg.tiles_per_image) { b0 = (int)(nt / cfg.tiles_per_image); h0 = (int)(nt % cfg.tiles_per_image) * cfg.th; }
                else { b0 = (int)(nt * cfg.tb); h0 = 0; }
                for (int kb = 0; kb < cfg.nkb; ++kb, ++g) {
                    const int s = g % kStages;
                    if (!mbar_wait(bar_empty + 8 * s, ((g / kStages) & 1) ^ 1, abort_flag)) break;
                    const int tap = kb / cfg.cpt, c0 = (kb - tap * cfg.cpt) * 128;
                    const int ti = tap / taps_w, tj = tap - ti * taps_w;
                    mbar_arrive_expect_tx(bar_full + 8 * s, cfg.tx_bytes);
                    tma_load_4d(sB + s * kBBytes, &act_map, bar_full + 8 * s, c0, tj - p.pad,
                                h0 * p.stride + ti - p.pad, b0);
                }
            }
            if (*abort_flag) {
                // give copies already in flight time to land before the CTA's memory is released
                for (int i = 0; i < 200; ++i) __nanosleep(1000);
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------- MMA issuer
        if (lane == 0) {
            uint32_t g = 0, it = 0;
            for (int64_t tile = first; tile < cfg.ntiles && !*abort_flag; tile += step, ++it) {
                const uint32_t ab = it & 1;
                if (!mbar_wait(bar_tempty + 8 * ab, ((it >> 1) & 1) ^ 1, abort_flag)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + ab * kTileN;
                bool ok = true;
                for (int kb = 0; kb < cfg.nkb; ++kb, ++g) {
                    const int s = g % kStages;
                    if (!mbar_wait(bar_full + 8 * s, (g / kStages) & 1, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const int c0 = (kb % cfg.cpt) * 128;
                    const int ksteps = (min(128, p.Cin - c0) + 31) >> 5;
                    const uint64_t ad = smem_desc_sw128(sA + s * kABytes), bd = smem_desc_sw128(sB + s * kBBytes);
                    for (int ks = 0; ks < ksteps; ++ks)
                        mma_i8(d_tmem, ad + 2 * ks, bd + 2 * ks, cfg.idesc, (kb | ks) ? 1u : 0u);
                    mma_commit(bar_empty + 8 * s);
                }
                if (!ok) break;
                mma_commit(bar_tfull + 8 * ab);
            }
        }
    } else if (warp < 2 + kNumExpWarps) {
        // ---------------------------------------------------------- expanders
        const int et = threadIdx.x - 64;          // 0..255
        const int q = et & 3;                     // k-step (32 codes) handled within each k-block
        const int slot0 = et >> 2;                // rows slot0 and slot0 + 64 of the tile's sorted order
        RowTask cur[2], nxt[2];
        int64_t load_tile = first;                // tile the load cursor is in
        cur[0] = make_task(p, load_tile < cfg.ntiles ? load_tile : -1, slot0);
        cur[1] = make_task(p, load_tile < cfg.ntiles ? load_tile : -1, slot0 + 64);
        {
            const int64_t t2 = load_tile + step;
            nxt[0] = make_task(p, t2 < cfg.ntiles ? t2 : -1, slot0);
            nxt[1] = make_task(p, t2 < cfg.ntiles ? t2 : -1, slot0 + 64);
        }
        int load_kb = 0;
        // k-blocks left for this CTA
        int64_t my_tiles = (cfg.ntiles > first) ? (cfg.ntiles - first + step - 1) / step : 0;
        const int64_t total = my_tiles * cfg.nkb;

        auto issue_load = [&](RawBuf& r, int64_t gl) {
            // load cursor -> registers, then advance the cursor
            if (gl >= total) { r.meta[0] = r.meta[1] = 3 << 8; return; }
            const int tap = load_kb / cfg.cpt, c0 = (load_kb - tap * cfg.cpt) * 128;
            const int ksteps = (min(128, p.Cin - c0) + 31) >> 5;
            exp_load(r, cur, tap * p.Cp + c0 + q * 32, q < ksteps);
            if (++load_kb == cfg.nkb) {
                load_kb = 0;
                load_tile += step;
                cur[0] = nxt[0]; cur[1] = nxt[1];
                const int64_t t2 = load_tile + step;
                nxt[0] = make_task(p, t2 < cfg.ntiles ? t2 : -1, slot0);
                nxt[1] = make_task(p, t2 < cfg.ntiles ? t2 : -1, slot0 + 64);
            }
        };
        bool alive = true;
        auto consume = [&](const RawBuf& r, int64_t g) {
            const int s = (int)(g % kStages);
            if (!mbar_wait_warp(bar_empty + 8 * s, (uint32_t)((g / kStages) & 1) ^ 1u, abort_flag)) { alive = false; return; }
            exp_store(r, sA + s * kABytes, q);
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_full + 8 * s);
        };

        RawBuf r0, r1, r2;
        issue_load(r0, 0);
        issue_load(r1, 1);
        for (int64_t g = 0; g < total && alive; g += 3) {
            issue_load(r2, g + 2);
            consume(r0, g);
            if (g + 1 < total) { issue_load(r0, g + 3); consume(r1, g + 1); }
            if (g + 2 < total) { issue_load(r1, g + 4); consume(r2, g + 2); }
        }
    } else {
        // ---------------------------------------------------------- epilogue
        const int quarter = warp & 3;              // TMEM lanes this warp may read
        const int half = (warp - (2 + kNumExpWarps)) >> 2;   // which chunks of a tile: even or odd
        uint32_t it = 0;
        for (int64_t tile = first; tile < cfg.ntiles; tile += step, ++it) {
            const uint32_t ab = it & 1;
            const int blk = (int)(tile % p.nblocks);
            const int64_t nt = tile / p.nblocks;
            int64_t n0;
            if (cfg.tiles_per_image) n0 = ((nt / cfg.tiles_per_image) * p.Ho + (nt % cfg.tiles_per_image) * cfg.th) * (int64_t)p.Wo;
            else n0 = nt * (int64_t)cfg.npix;
            const int nvalid = (int)min((int64_t)cfg.npix, p.N - n0);
            const int m = blk * kBlockRows + quarter * 32 + lane;
            const bool row_ok = m < p.M;
            float scale = 0.f;
            int shift = 0;
            if (row_ok) {
                scale = __fmul_rn(__ldg(p.wstep + m), p.act_step);
                shift = (__ldg(p.kind + m) == kFixed4) ? 4 : 0;
            }
            if (!mbar_wait_warp(bar_tfull + 8 * ab, (it >> 1) & 1, abort_flag)) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + ab * kTileN;
            if (cfg.tma_store) {
                // The warps of a tensor-memory quarter take alternate 32-pixel chunks of its 32 rows; each
                // stages its chunk in a private buffer and issues its own bulk store, so no epilogue
                // warp ever waits for another.
                if (blk * kBlockRows + quarter * 32 >= p.M) {      // no valid row in this quarter
                    tc_fence_before();
                    if (lane == 0) mbar_arrive(bar_tempty + 8 * ab);
                    continue;
                }
                const uint32_t stg = sOut + (uint32_t)(warp - (2 + kNumExpWarps)) * kWarpStage;
                const int nchunks = (nvalid + 31) >> 5;
                if (half >= nchunks) {                             // a one-chunk tile leaves the odd warps idle
                    tc_fence_before();
                    if (lane == 0) mbar_arrive(bar_tempty + 8 * ab);
                    continue;
                }
                for (int c = half; c < nchunks; c += kEpiPerQuarter) {
                    uint32_t v[32];
                    tmem_ld32(taddr + c * 32, v);
                    if (c + kEpiPerQuarter >= nchunks) {
                        // all accumulators of this tile are in registers: hand the buffer back
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar_tempty + 8 * ab);
                    }
                    const bool tail = cfg.tail_rows && (c == (cfg.npix >> 5));
                    const int nsub = p.acc ? 2 : 1;
                    for (int sub = 0; sub < nsub; ++sub) {
                        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                        __syncwarp();                    // the buffer's previous store has been read out
                        if (!p.out_mn) {
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
                            for (int cc = 0; cc < 8; ++cc) {
                                uint32_t w[4];
#pragma unroll
                                for (int t = 0; t < 4; ++t) {
                                    const int a = (int)v[4 * cc + t] >> shift;
                                    w[t] = sub ? (uint32_t)a : __float_as_uint(__fmul_rn(__int2float_rn(a), scale));
                                }
                                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                                             ::"r"(a0 + ((cc ^ (lane & 7)) << 4)), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
                            }
                        }
                        fence_proxy_async_smem();
                        __syncwarp();                    // chunk complete in shared memory
                        if (lane == 0) {
                            const CUtensorMap* map = sub ? (tail ? &smaps.acc_tail : &smaps.acc_full)
                                                         : (tail ? &smaps.out_tail : &smaps.out_full);
                            const int cm = blk * kBlockRows + quarter * 32, cn = (int)(n0 + c * 32);
                            if (!p.out_mn) tma_store_2d(map, stg, cm, cn); else tma_store_2d(map, stg, cn, cm);
                        }
                    }
                }
                continue;
            }
            for (int c = 0; c * 32 < nvalid; ++c) {
                uint32_t v[32];
                tmem_ld32(taddr + c * 32, v);
                const int jmax = min(32, nvalid - c * 32);
                if (row_ok) {
                    if (!p.out_mn) {
                        float* o = p.out + (n0 + c * 32) * p.ld_out + m;
                        int32_t* oa = p.acc ? p.acc + (n0 + c * 32) * p.ld_out + m : nullptr;
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
                        int32_t* oa = p.acc ? p.acc + (int64_t)m * p.ld_out + n0 + c * 32 : nullptr;
                        const bool vec = (jmax == 32) && ((reinterpret_cast<uintptr_t>(o) & 15) == 0);
                        if (vec) {
#pragma unroll
                            for (int j = 0; j < 32; j += 4) {
                                float4 f;
                                f.x = __fmul_rn(__int2float_rn((int)v[j] >> shift), scale);
                                f.y = __fmul_rn(__int2float_rn((int)v[j + 1] >> shift), scale);
                                f.z = __fmul_rn(__int2float_rn((int)v[j + 2] >> shift), scale);
                                f.w = __fmul_rn(__int2float_rn((int)v[j + 3] >> shift), scale);
                                *reinterpret_cast<float4*>(o + j) = f;
                                if (oa) *reinterpret_cast<int4*>(oa + j) = make_int4((int)v[j] >> shift, (int)v[j + 1] >> shift,
                                                                                     (int)v[j + 2] >> shift, (int)v[j + 3] >> shift);
                            }
                        } else {
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
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_tempty + 8 * ab);
        }
    }

    // ---------------------------------------------------------- teardown
    if (warp >= 2 + kNumExpWarps && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
    }
    if (threadIdx.x == 0 && s_abort) atomicMax(p.status, (uint32_t)RMSMP_ERR_TIMEOUT);
}

// ------------------------------------------------------------------ host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
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

bool plan(const Problem& p, TensorCfg& c)
{
    if (p.pix_pitch % 16 != 0 || p.Cin % 16 != 0) return false;
    if ((reinterpret_cast<uintptr_t>(p.act) & 15) != 0) return false;
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
    c.cpt = (p.Cin + 127) / 128;
    c.nkb = p.kh * p.kw * c.cpt;
    c.tx_bytes = (uint32_t)c.npix * 128u;
    // kind::i8: int32 accumulate (bits 4-5 = 2), signed 8-bit A and B (bits 7-9, 10-12 = 1),
    // both K-major, N/8 at bit 17, M/16 at bit 24
    c.idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(c.n_mma >> 3) << 17) | ((uint32_t)(kBlockRows >> 4) << 24);
    return true;
}

}  // namespace

bool tensor_supported(const Problem& p)
{
    TensorCfg c;
    return plan(p, c) && encode_fn() != nullptr;
}

rmsmp_status launch_tensor(const Problem& p, cudaStream_t st)
{
    TensorCfg c;
    if (!plan(p, c)) return RMSMP_ERR_VARIANT;
    EncodeTiledFn enc = encode_fn();
    if (!enc) return RMSMP_ERR_CUDA;
    CUtensorMap map;
    const cuuint64_t gdim[4] = {(cuuint64_t)p.Cin, (cuuint64_t)p.W, (cuuint64_t)p.H, (cuuint64_t)p.B};
    const cuuint64_t gstr[3] = {(cuuint64_t)p.pix_pitch, (cuuint64_t)p.pix_pitch * p.W,
                                (cuuint64_t)p.pix_pitch * p.W * p.H};
    const cuuint32_t box[4] = {128u, (cuuint32_t)(p.Wo * p.stride), (cuuint32_t)(c.th * p.stride), (cuuint32_t)c.tb};
    const cuuint32_t estr[4] = {1u, (cuuint32_t)p.stride, (cuuint32_t)p.stride, 1u};
    CUresult r = enc(&map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<int8_t*>(p.act), gdim, gstr, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return RMSMP_ERR_CUDA;

    StoreMaps sm;
    memset(&sm, 0, sizeof(sm));
    c.tma_store = 0;
    c.tail_rows = c.npix & 31;
    const bool ld_ok = (p.ld_out % 4 == 0) && ((reinterpret_cast<uintptr_t>(p.out) & 15) == 0) &&
                       (!p.acc || (reinterpret_cast<uintptr_t>(p.acc) & 15) == 0);
    if (ld_ok && (!p.out_mn || c.tail_rows == 0)) {
        auto make = [&](CUtensorMap* m, void* base, CUtensorMapDataType dt, int rows) -> bool {
            if (!p.out_mn) {
                const cuuint64_t gd[2] = {(cuuint64_t)p.M, (cuuint64_t)p.N};
                const cuuint64_t gs[1] = {(cuuint64_t)p.ld_out * 4};
                const cuuint32_t bx[2] = {32u, (cuuint32_t)rows};
                const cuuint32_t es[2] = {1, 1};
                return enc(m, dt, 2, base, gd, gs, bx, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                           CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
            }
            const cuuint64_t gd[2] = {(cuuint64_t)p.N, (cuuint64_t)p.M};
            const cuuint64_t gs[1] = {(cuuint64_t)p.ld_out * 4};
            const cuuint32_t bx[2] = {32u, 32u};
            const cuuint32_t es[2] = {1, 1};
            return enc(m, dt, 2, base, gd, gs, bx, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                       CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
        };
        bool ok = make(&sm.out_full, p.out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 32);
        if (ok && c.tail_rows) ok = make(&sm.out_tail, p.out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, c.tail_rows);
        if (ok && p.acc) ok = make(&sm.acc_full, p.acc, CU_TENSOR_MAP_DATA_TYPE_INT32, 32);
        if (ok && p.acc && c.tail_rows) ok = make(&sm.acc_tail, p.acc, CU_TENSOR_MAP_DATA_TYPE_INT32, c.tail_rows);
        c.tma_store = ok ? 1 : 0;
    }

    static int sm_count = 0;
    static bool attr_set = false;
    if (!attr_set) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev);
        if (cudaFuncSetAttribute(tensor_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess) {
            cudaGetLastError();
            return RMSMP_ERR_CUDA;
        }
        attr_set = true;
    }
    const int grid = (int)std::min<int64_t>(c.ntiles, sm_count > 0 ? sm_count : 148);
    tensor_kernel<<<grid, kThreads, kSmemBytes, st>>>(p, c, map, sm);
    if (cudaGetLastError() != cudaSuccess) return RMSMP_ERR_CUDA;
    return RMSMP_OK;
}

}  // namespace rmsmp
