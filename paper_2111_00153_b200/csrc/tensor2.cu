// Pair kernel of the workspace mode: two CTAs of a cluster work on ONE output tile of 256 weight
// rows x up to 256 pixels with tcgen05.mma.cta_group::2.
//
// Why: a single CTA reads both MMA operands from its shared memory (12 KB per 128x256x32
// instruction, 96 B/clk at the pipe's full rate) while TMA refills the stages through the same
// 128 B/clk port, so it cannot keep the tensor pipe full.  In a pair each CTA holds its own 128
// weight rows and HALF of the pixels; the hardware feeds both tensor cores from both halves, so
// per instruction a CTA reads 8 KB and receives 8 KB.
//
// Roles per CTA (448 threads): warp 0 lane 0 fetches this CTA's half of the activation codes,
// warp 2 lane 0 its 128 expanded weight rows (both signal the LEADER's "full" barrier, rank 0;
// warps 3 and 4 are second producers taking the odd k-blocks),
// warp 1 of the leader issues the MMAs and commits to both CTAs' barriers, warps 6-13 are the
// epilogue of this CTA's 128 rows (tcgen05.ld, scale, staged bulk stores as in the single-CTA
// kernel).  Accumulators: tensor-memory columns [0, N) and [256, 256 + N), alternating by tile.
// A tile's pixels are two "halves" of up to 128 pixels each (whole images, or whole output rows of
// one image); half h occupies accumulator columns h * nh_pad ...
//
// Every mbarrier wait is bounded; when one runs out the CTA records RMSMP_ERR_TIMEOUT, its roles
// leave their loops and both CTAs still meet at the closing cluster barrier, free tensor memory
// and return.  No load uses cluster multicast.
#include <cuda.h>
#include <cstring>
#include <algorithm>
#include "common.cuh"

namespace rmsmp {

namespace {

constexpr int kThreads2 = 448;
constexpr int kStageA = 128 * 128;               // 16 KB: 128 rows x 128 B
constexpr int kStageB = 128 * 128;               // 16 KB: up to 128 pixels x 128 B
constexpr int kWarpStage2 = 32 * 32 * 4;         // per-warp output staging
constexpr int kEpiWarps2 = 8;
constexpr int kFirstEpi2 = 6;                   // warps 6-13, two per tensor-memory quarter
constexpr int kRing2 = 3;                       // stages; a stage holds TWO k-blocks of each operand (64 KB per CTA)
constexpr int kSub2 = 2;
constexpr long long kWaitCycles2 = 2000000000LL;

struct PairCfg {
    int tb, th;              // images / output rows per half
    int npix_h;              // pixels per half
    int nh_pad;              // npix_h rounded up to 8: accumulator columns per half
    int halves_per_image;    // Ho/th when tb == 1 and th < Ho, else 0
    int64_t nhalves;         // halves in the problem
    int64_t ntiles_n;        // pixel tiles = ceil(nhalves / 2)
    int nbt;                 // row-block pairs
    int64_t ntiles;          // ntiles_n * nbt
    int cpt;                 // 128-channel chunks per tap
    int nkb;                 // k-blocks per tile
    uint32_t idesc;
    uint32_t tx_b;           // bytes one activation box brings
    int tail_rows;           // npix_h % 32
    uint32_t smem_bytes;
};

struct PairMaps {
    CUtensorMap act[4], wexp, out_full, out_tail;      // act: one map, or one per parity sub-grid (stride 2)
};

__device__ __forceinline__ uint32_t s32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint32_t cluster_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of `addr` (a shared::cta address of this CTA) in CTA `rank`
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void bar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
// arrivals on a barrier given by its shared::cluster address (own or peer CTA)
__device__ __forceinline__ void bar_arrive_cluster(uint32_t cbar)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cbar) : "memory");
}
__device__ __forceinline__ bool bar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool bar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag)
{
    if (bar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 64; ++i)
            if (bar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > kWaitCycles2) { *abort_flag = 1; return false; }
    }
}
__device__ __forceinline__ bool bar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag)
{
    bool ok = true;
    if ((threadIdx.x & 31) == 0) ok = bar_wait(bar, parity, abort_flag);
    return __all_sync(0xffffffffu, ok);
}
// TMA loads of a CTA pair: data into this CTA's shared memory, completion on a barrier that may
// live in the peer CTA (cta_group::2 form; no multicast).
__device__ __forceinline__ void pair_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t cbar, int c0, int c1, int c2, int c3)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(map), "r"(cbar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void pair_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t cbar, int c0, int c1)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(cbar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void store_2d(const CUtensorMap* map, uint32_t src, int c0, int c1)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(map), "r"(src), "r"(c0), "r"(c1) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// One MMA of the pair: 256 rows (128 per CTA) x N columns x 32 codes; descriptors as 32-bit halves.
__device__ __forceinline__ void pair_mma(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "mov.b64 da, {%1, %3};\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], da, db, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrive (once all MMAs issued so far have finished) on the barrier at this shared-memory offset in BOTH CTAs.
__device__ __forceinline__ void pair_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((uint16_t)3) : "memory");
}
__device__ __forceinline__ void ld_issue(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void ld_wait(uint32_t (&v)[32])
{
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]),
                   "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15]),
                   "+r"(v[16]), "+r"(v[17]), "+r"(v[18]), "+r"(v[19]), "+r"(v[20]), "+r"(v[21]), "+r"(v[22]), "+r"(v[23]),
                   "+r"(v[24]), "+r"(v[25]), "+r"(v[26]), "+r"(v[27]), "+r"(v[28]), "+r"(v[29]), "+r"(v[30]), "+r"(v[31])
                 :: "memory");
}

// First pixel and geometry of half `hf` (global half index): image / row coordinates for the TMA
// box and the index of its first output pixel.
struct HalfPos { int b0, h0; int64_t n0; };
__device__ __forceinline__ HalfPos half_pos(const Problem& p, const PairCfg& cfg, int64_t hf)
{
    HalfPos r;
    if (cfg.halves_per_image) {
        r.b0 = (int)(hf / cfg.halves_per_image);
        r.h0 = (int)(hf - (int64_t)r.b0 * cfg.halves_per_image) * cfg.th;
        r.n0 = ((int64_t)r.b0 * p.Ho + r.h0) * p.Wo;
    } else {
        r.b0 = (int)(hf * cfg.tb);
        r.h0 = 0;
        r.n0 = hf * (int64_t)cfg.npix_h;
    }
    return r;
}

__global__ void __launch_bounds__(kThreads2, 1)
pair_kernel(const Problem p, const PairCfg cfg, const __grid_constant__ PairMaps maps)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (s32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sA = smem_base;
    const uint32_t sB = sA + kRing2 * kSub2 * kStageA;
    const uint32_t sOut = sB + kRing2 * kSub2 * kStageB;
    const uint32_t sBar = sOut + kEpiWarps2 * kWarpStage2;
    const uint32_t bar_full = sBar, bar_empty = sBar + 8 * kRing2;
    const uint32_t bar_tfull = sBar + 16 * kRing2, bar_tempty = bar_tfull + 16;
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();                 // 0 = leader: owns the "full" and "accumulator free" barriers

    if (threadIdx.x == 0) {
        for (int s = 0; s < kRing2; ++s) {
            bar_init(bar_full + 8 * s, 1);       // the leader's activation producer announces all four copies' bytes; leader only
            bar_init(bar_empty + 8 * s, 1);      // the leader's commit, delivered to both CTAs
        }
        for (int b = 0; b < 2; ++b) {
            bar_init(bar_tfull + 8 * b, 1);                    // the leader's commit, delivered to both CTAs
            bar_init(bar_tempty + 8 * b, 2 * kEpiWarps2);      // every epilogue warp of both CTAs; used in the leader only
        }
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        // one warp of EACH CTA of the pair takes part in the allocation
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(s32(&s_tmem_base)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    cluster_sync_all();                                   // both CTAs' barriers exist before anyone signals the peer
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = s_tmem_base;
    volatile int* abort_flag = &s_abort;

    const int64_t first = blockIdx.x >> 1, step = gridDim.x >> 1;      // cluster index, clusters in the grid
    const uint32_t lead_full = map_to_rank(bar_full, 0), lead_tempty = map_to_rank(bar_tempty, 0);

    if (warp == 0 || warp == 2 || warp == 3 || warp == 4) {
      if (lane == 0) {
        // ---------------------------------------------------------- producers (both CTAs)
        // One thread can start a bulk tensor copy only every ~300 ns, about the time four MMAs take,
        // so each operand has two producer threads taking alternate stages.
        const bool is_b = (warp == 0 || warp == 3);
        const uint32_t mine = (warp >= 3) ? 1u : 0u;
        uint32_t s = 0, ph = 0, g = 0;
        bool ok = true;
        for (int64_t tile = first; tile < cfg.ntiles && ok; tile += step) {
            const int64_t nt = tile / cfg.nbt;
            const int blk = (int)(tile - nt * cfg.nbt) * 2 + (int)rank;        // this CTA's row block
            const HalfPos hp = half_pos(p, cfg, 2 * nt + rank);               // this CTA's half of the pixels
            int tap = 0, cc = 0, ti = 0, tj = 0;
            for (int kb = 0; kb < cfg.nkb; kb += kSub2, ++g) {
                const int nsub = min(kSub2, cfg.nkb - kb);
                const bool skip = (g & 1u) != mine;
                if (!skip) {
                    if (!bar_wait(bar_empty + 8 * s, ph ^ 1, abort_flag)) { ok = false; break; }
                    // all copies of this stage (up to two k-blocks of two operands in two CTAs) complete on the leader's barrier
                    if (is_b && rank == 0)
                        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                                     ::"r"(bar_full + 8 * s), "r"(2u * nsub * (cfg.tx_b + (uint32_t)kStageA)) : "memory");
                }
                const uint32_t fb = lead_full + 8 * s;
                for (int u = 0; u < nsub; ++u) {
                    if (!skip) {
                        if (is_b) {
                            const TapBox tb = tap_box(p, hp.h0, ti, tj);
                            pair_load_4d(sB + (s * kSub2 + u) * kStageB, &maps.act[tb.map], fb, cc * 128, tb.x, tb.y, hp.b0);
                        }
                        else pair_load_2d(sA + (s * kSub2 + u) * kStageA, &maps.wexp, fb, tap * p.Cp + cc * 128, blk * kBlockRows);
                    }
                    if (++cc == cfg.cpt) { cc = 0; ++tap; if (++tj == p.kw) { tj = 0; ++ti; } }
                }
                if (++s == kRing2) { s = 0; ph ^= 1; }
            }
        }
        if (!ok) {
            for (int i = 0; i < 200; ++i) __nanosleep(1000);   // let copies in flight land
        }
      }
    } else if (warp == 1) {
        // ---------------------------------------------------------- MMA issuer (leader CTA only)
        if (rank == 0) {
            const bool issuer = (lane == 0);
            uint32_t s = 0, ph = 0, it = 0;
            const uint32_t hi = (uint32_t)(1024 >> 4) | (1u << 14) | (2u << 29);     // SBO 1024 B, version 1, 128-byte swizzle
            const uint32_t a_lo0 = ((sA >> 4) & 0x3FFFu) | (1u << 16), b_lo0 = ((sB >> 4) & 0x3FFFu) | (1u << 16);
            const uint32_t a_step = (kSub2 * kStageA) >> 4, b_step = (kSub2 * kStageB) >> 4;
            uint32_t a_lo = a_lo0, b_lo = b_lo0;
            for (int64_t tile = first; tile < cfg.ntiles && !*abort_flag; tile += step, ++it) {
                const uint32_t ab = it & 1;
                if (!bar_wait(bar_tempty + 8 * ab, ((it >> 1) & 1) ^ 1, abort_flag)) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t d_tmem = tmem_base + ab * 256;
                bool ok = true;
                for (int kb = 0; kb < cfg.nkb; kb += kSub2) {
                    if (!bar_wait(bar_full + 8 * s, ph, abort_flag)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    if (issuer) {
                        pair_mma(d_tmem, a_lo, b_lo, hi, cfg.idesc, kb ? 1u : 0u);
                        pair_mma(d_tmem, a_lo + 2, b_lo + 2, hi, cfg.idesc, 1u);
                        pair_mma(d_tmem, a_lo + 4, b_lo + 4, hi, cfg.idesc, 1u);
                        pair_mma(d_tmem, a_lo + 6, b_lo + 6, hi, cfg.idesc, 1u);
                        if (kb + 1 < cfg.nkb) {
                            const uint32_t a1 = a_lo + (kStageA >> 4), b1 = b_lo + (kStageB >> 4);
                            pair_mma(d_tmem, a1, b1, hi, cfg.idesc, 1u);
                            pair_mma(d_tmem, a1 + 2, b1 + 2, hi, cfg.idesc, 1u);
                            pair_mma(d_tmem, a1 + 4, b1 + 4, hi, cfg.idesc, 1u);
                            pair_mma(d_tmem, a1 + 6, b1 + 6, hi, cfg.idesc, 1u);
                        }
                        pair_commit(bar_empty + 8 * s);
                    }
                    a_lo += a_step;
                    b_lo += b_step;
                    if (++s == kRing2) { s = 0; ph ^= 1; a_lo = a_lo0; b_lo = b_lo0; }
                }
                if (!ok) break;
                if (issuer) pair_commit(bar_tfull + 8 * ab);
            }
        }
    } else if (warp >= kFirstEpi2) {
        // ---------------------------------------------------------- epilogue (both CTAs, own 128 rows)
        const int quarter = warp & 3;
        const int first_epi = kFirstEpi2;
        auto count_q = [&](int q) { const int f = first_epi + ((q - first_epi) & 3); return (kThreads2 / 32 - 1 - f) / 4 + 1; };
        const int my_rank = (warp - (first_epi + ((quarter - first_epi) & 3))) >> 2;
        const int cstride = count_q(quarter);
        const uint32_t my_stage = sOut + (uint32_t)(warp - first_epi) * kWarpStage2;
        const int nch = (cfg.npix_h + 31) >> 5;              // 32-pixel chunks per half
        uint32_t it = 0;
        bool alive = true;
        for (int64_t tile = first; tile < cfg.ntiles && alive; tile += step, ++it) {
            const uint32_t ab = it & 1;
            const int64_t nt = tile / cfg.nbt;
            const int blk = (int)(tile - nt * cfg.nbt) * 2 + (int)rank;
            const int m = blk * kBlockRows + quarter * 32 + lane;
            const float scale = (m < p.M) ? __fmul_rn(__ldg(p.wstep + m), p.act_step) : 0.f;
            int64_t n0h[2];
            int nvalid[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const HalfPos hp = half_pos(p, cfg, 2 * nt + h);
                n0h[h] = hp.n0;
                nvalid[h] = (int)max((int64_t)0, min((int64_t)cfg.npix_h, p.N - hp.n0));
            }
            if (!bar_wait_warp(bar_tfull + 8 * ab, (it >> 1) & 1, abort_flag)) { alive = false; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + ab * 256;
            const bool rows_ok = blk * kBlockRows + quarter * 32 < p.M;
            // chunk index i = h * nch + c; this warp takes i = my_rank, my_rank + cstride, ...
            uint32_t v[32];
            for (int i = my_rank; i < 2 * nch; i += cstride) {
                const int h = i >= nch, c = i - h * nch;
                if (!rows_ok || c * 32 >= nvalid[h]) continue;
                ld_issue(taddr + h * cfg.nh_pad + c * 32, v);
                ld_wait(v);
                if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                __syncwarp();
                const uint32_t a0 = my_stage + lane * 4;
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const uint32_t w = __float_as_uint(__fmul_rn(__int2float_rn((int)v[j]), scale));
                    asm volatile("st.shared.b32 [%0], %1;" ::"r"(a0 + j * 128), "r"(w) : "memory");
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) {
                    const bool tail = cfg.tail_rows && (c == (cfg.npix_h >> 5));
                    store_2d(tail ? &maps.out_tail : &maps.out_full, my_stage, blk * kBlockRows + quarter * 32, (int)(n0h[h] + c * 32));
                }
            }
            // accumulators of this tile are out of tensor memory: tell the leader
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) bar_arrive_cluster(lead_tempty + 8 * ab);
        }
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    }

    // ---------------------------------------------------------- teardown
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    cluster_sync_all();                                   // nobody signals a CTA that has left
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
    }
    if (threadIdx.x == 0 && s_abort) atomicMax(p.status, (uint32_t)RMSMP_ERR_TIMEOUT);
}

// ------------------------------------------------------------------ host side

typedef CUresult (*EncodeTiledFn2)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                   CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                   CUtensorMapFloatOOBfill);

EncodeTiledFn2 encode_fn2()
{
    static EncodeTiledFn2 fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn2>(ptr);
        else
            cudaGetLastError();
    }
    return fn;
}

// The pair kernel takes: expanded weights, an even number of row blocks, full 128-channel chunks,
// fp32 [N][M] output through bulk stores, no accumulator dump, no re-quantizing epilogue.
bool plan_pair(const Problem& p, PairCfg& c)
{
    if (!p.wexp || p.acc || p.rq_codes || p.out_mn) return false;
    if (p.nblocks < 2 || (p.nblocks & 1)) return false;
    if (p.Cin % 128 != 0 || p.pix_pitch % 16 != 0) return false;
    if ((reinterpret_cast<uintptr_t>(p.act) & 15) || (reinterpret_cast<uintptr_t>(p.wexp) & 15)) return false;
    if ((p.ld_out % 4) || (p.M % 4) || (reinterpret_cast<uintptr_t>(p.out) & 15)) return false;
    const int64_t hw = (int64_t)p.Ho * p.Wo;
    if (p.Wo > 128 || (int64_t)p.Wo * p.stride > 256) return false;
    if (hw <= 128) {
        c.th = p.Ho;
        c.tb = (int)std::min<int64_t>(128 / hw, p.B);
        c.halves_per_image = 0;
        c.nhalves = (p.B + c.tb - 1) / c.tb;
    } else {
        int th = 1;
        for (int d = 1; d <= p.Ho; ++d)
            if (p.Ho % d == 0 && (int64_t)d * p.Wo <= 128) th = d;
        c.th = th; c.tb = 1;
        c.halves_per_image = p.Ho / th;
        c.nhalves = (int64_t)p.B * c.halves_per_image;
    }
    if ((int64_t)c.th * p.stride > 256) return false;
    c.npix_h = c.tb * c.th * p.Wo;
    c.nh_pad = (c.npix_h + 7) / 8 * 8;
    c.ntiles_n = (c.nhalves + 1) / 2;
    c.nbt = p.nblocks / 2;
    c.ntiles = c.ntiles_n * c.nbt;
    c.cpt = p.Cin / 128;
    c.nkb = p.kh * p.kw * c.cpt;
    c.tx_b = (uint32_t)c.npix_h * 128u;
    c.tail_rows = c.npix_h & 31;
    // kind::i8, int32 accumulate, signed 8-bit A and B, K-major; N = both halves, M = 256 over the pair
    c.idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)((2 * c.nh_pad) >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
    c.smem_bytes = (uint32_t)(kRing2 * kSub2 * (kStageA + kStageB) + kEpiWarps2 * kWarpStage2 + 1024 + 64 * 2 * kRing2);
    return true;
}

}  // namespace

// Worth it when K is long (short reductions are dominated by the pair's start-up and by the
// epilogue: BERT-base FFN1 with 6 k-blocks is 40 % slower this way) and both halves are well filled.
bool pair_supported(const Problem& p)
{
    PairCfg c;
    if (!plan_pair(p, c) || !encode_fn2()) return false;
    return c.nkb >= 16 && c.npix_h >= 64;
}

rmsmp_status launch_pair(const Problem& p, cudaStream_t st)
{
    PairCfg c;
    if (!plan_pair(p, c)) return RMSMP_ERR_VARIANT;
    EncodeTiledFn2 enc = encode_fn2();
    if (!enc) return RMSMP_ERR_CUDA;
    PairMaps mp;
    memset(&mp, 0, sizeof(mp));
    if (!encode_act_maps_4(p, 128, c.th, c.tb, mp.act)) return RMSMP_ERR_CUDA;
    {
        const cuuint64_t gd[2] = {(cuuint64_t)p.Kp, (cuuint64_t)p.M};
        const cuuint64_t gs[1] = {(cuuint64_t)p.Kp};
        const cuuint32_t bx[2] = {128u, (cuuint32_t)kBlockRows};
        const cuuint32_t es[2] = {1, 1};
        if (enc(&mp.wexp, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t*>(p.wexp), gd, gs, bx, es,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return RMSMP_ERR_CUDA;
    }
    auto make_out = [&](CUtensorMap* m, int rows) -> bool {
        const cuuint32_t es[2] = {1, 1};
        const cuuint64_t gs[1] = {(cuuint64_t)p.ld_out * 4};
        const cuuint64_t gd[2] = {(cuuint64_t)p.M, (cuuint64_t)p.N};
        const cuuint32_t bx[2] = {32u, (cuuint32_t)rows};
        return enc(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, p.out, gd, gs, bx, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    };
    if (!make_out(&mp.out_full, 32)) return RMSMP_ERR_CUDA;
    if (c.tail_rows && !make_out(&mp.out_tail, c.tail_rows)) return RMSMP_ERR_CUDA;

    static bool attr_set[kMaxDevices] = {};
    if (!ensure_smem_attr(reinterpret_cast<const void*>(pair_kernel), (int)c.smem_bytes, attr_set)) return RMSMP_ERR_CUDA;
    const int clusters = (int)std::min<int64_t>(c.ntiles, sm_count() / 2);
    cudaLaunchConfig_t lc;
    memset(&lc, 0, sizeof(lc));
    lc.gridDim = dim3((unsigned)(2 * clusters), 1, 1);
    lc.blockDim = dim3(kThreads2, 1, 1);
    lc.dynamicSmemBytes = c.smem_bytes;
    lc.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    lc.attrs = at;
    lc.numAttrs = 1;
    if (cudaLaunchKernelEx(&lc, pair_kernel, p, c, mp) != cudaSuccess) {
        cudaGetLastError();
        return RMSMP_ERR_CUDA;
    }
    return RMSMP_OK;
}

}  // namespace rmsmp
