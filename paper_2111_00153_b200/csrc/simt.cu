// CUDA-core variants of the contraction: a one-thread-per-output cross-check kernel and a
// row-per-warp kernel (integer dot products on codes expanded in registers, or -- for PoT
// rows -- shifts and adds without a multiplier).
#include <cstring>
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
    if (blocks > (int64_t)sm_count() * 64) blocks = (int64_t)sm_count() * 64;
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
    if (blocks > (int64_t)sm_count() * 8) blocks = (int64_t)sm_count() * 8;
    if (shiftadd) rowwarp_kernel<true><<<(unsigned)blocks, 256, 0, st>>>(p);
    else rowwarp_kernel<false><<<(unsigned)blocks, 256, 0, st>>>(p);
    return cudaGetLastError();
}

// ------------------------------------------------------------------ grouped small-batch launch
// Many weight-bound linear layers (a few tokens each) in ONE launch: with one launch per layer
// the few hundred nanoseconds the weights need at HBM speed disappear behind launch latency.
// The table in device memory holds the problems and the running count of work items; a work
// item is (problem, up to RW consecutive packed rows of ONE kind, group of NT tokens), so the
// row loop of an item has no per-row branches.  A warp keeps the 16-byte chunks of its RW rows
// in flight together, so enough bytes are outstanding per SM to stream the packed weights at
// memory speed.  Each block first copies the table to shared memory (when it fits), which takes
// the table look-ups out of the dependent-load chain in front of every item's weight loads.

struct GroupedTable {          // device layout: header, cum[count + 1], then Problem[count] at `prob_off`
    int32_t count;
    int32_t prob_off;          // bytes from the table start
    int64_t total;             // work items
    int32_t bytes;             // whole table
    int32_t pad;
};

constexpr int kGroupedSmemMax = 96 * 1024;

__host__ __device__ inline int grouped_rw(int kind, int nt)
{
    if (nt == 1) return kind == kFixed8 ? 4 : 8;
    return kind == kFixed8 ? 2 : 4;
}

template <int KIND>
__device__ __forceinline__ void grouped_expand(const uint4& lo, const uint4& hi, uint32_t wv[8])
{
    if (KIND == kFixed8) {
        wv[0] = lo.x; wv[1] = lo.y; wv[2] = lo.z; wv[3] = lo.w;
        wv[4] = hi.x; wv[5] = hi.y; wv[6] = hi.z; wv[7] = hi.w;
    } else if (KIND == kPoT4) {
        expand_pot_chunk(lo, wv);
    } else {
        expand_fixed4_chunk_x16(lo, wv);
    }
}

template <int KIND, int NT, int RW>
__device__ __forceinline__ void grouped_rows(const Problem& p, int pr0, int nrows, int64_t n0, int lane)
{
    const int n4 = p.nP + p.nF4;
    const int nchunks = p.Cp >> 5;                           // linear layers: one tap
    const size_t pitch = (KIND == kFixed8) ? (size_t)p.Kp : (size_t)(p.Kp >> 1);
    const uint8_t* base = (KIND == kFixed8) ? p.q8 + (size_t)(pr0 - n4) * pitch : p.q4 + (size_t)pr0 * pitch;
    // Lane r fetches row r's original index and scale now, so that these two dependent loads
    // overlap the weight stream instead of following it.
    int row_m = 0;
    float row_c = 0.0f;
    if (lane < nrows) {
        row_m = p.perm[pr0 + lane];
        row_c = __fmul_rn(p.wstep[row_m], p.act_step);
    }
    int acc[RW][NT];
#pragma unroll
    for (int r = 0; r < RW; ++r)
#pragma unroll
        for (int t = 0; t < NT; ++t) acc[r][t] = 0;
    for (int ch = lane; ch < nchunks; ch += 32) {
        const int kp = ch << 5;
        const size_t off = (KIND == kFixed8) ? (size_t)kp : (size_t)(kp >> 1);
        uint4 raw[RW], raw2[KIND == kFixed8 ? RW : 1];
#pragma unroll
        for (int r = 0; r < RW; ++r) {                       // all rows' loads in flight together
            const int rr = r < nrows ? r : nrows - 1;        // rows past the item's end repeat its last one
            const uint4* src = reinterpret_cast<const uint4*>(base + (size_t)rr * pitch + off);
            raw[r] = __ldcs(src);
            if (KIND == kFixed8) raw2[r] = __ldcs(src + 1);
        }
        const bool full = (kp + 32 <= p.Cin);
        // One token: its codes are loaded once and each row is expanded right before its dot
        // product.  Several tokens: all rows are expanded first, then tokens stream through.
        uint32_t wv[NT == 1 ? 1 : RW][8];
        if (NT > 1) {
#pragma unroll
            for (int r = 0; r < RW; ++r) grouped_expand<KIND>(raw[r], raw2[KIND == kFixed8 ? r : 0], wv[NT == 1 ? 0 : r]);
        }
#pragma unroll
        for (int t = 0; t < NT; ++t) {
            const int64_t n = (n0 + t < p.N) ? n0 + t : p.N - 1;
            const int8_t* ap = p.act + n * p.pix_pitch + kp;
            uint32_t a[8];
            if (full) {
                const uint4 lo = __ldg(reinterpret_cast<const uint4*>(ap)), hi = __ldg(reinterpret_cast<const uint4*>(ap) + 1);
                a[0] = lo.x; a[1] = lo.y; a[2] = lo.z; a[3] = lo.w;
                a[4] = hi.x; a[5] = hi.y; a[6] = hi.z; a[7] = hi.w;
            } else {
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    uint32_t v = 0;
#pragma unroll
                    for (int bb = 0; bb < 4; ++bb)
                        if (kp + q * 4 + bb < p.Cin) v |= (uint32_t)(uint8_t)ap[q * 4 + bb] << (8 * bb);
                    a[q] = v;
                }
            }
#pragma unroll
            for (int r = 0; r < RW; ++r) {
                if (NT == 1) {
                    grouped_expand<KIND>(raw[r], raw2[KIND == kFixed8 ? r : 0], wv[0]);
                    acc[r][t] = dot32(wv[0], a, acc[r][t]);
                } else {
                    acc[r][t] = dot32(wv[NT == 1 ? 0 : r], a, acc[r][t]);
                }
            }
        }
    }
    // Lane r*NT + t finishes element (row r, token t) with the row data lane r fetched up front.
    int mine = 0;
#pragma unroll
    for (int r = 0; r < RW; ++r)
#pragma unroll
        for (int t = 0; t < NT; ++t) {
            int v = __reduce_add_sync(0xffffffffu, acc[r][t]);
            if (KIND == kFixed4) v >>= 4;                    // the Fixed-4 codes were expanded as 16 * value
            if (lane == r * NT + t) mine = v;
        }
    static_assert(RW * NT <= 32, "one lane per element of a work item");
    const int er = lane / NT, et = lane % NT;
    const int m = __shfl_sync(0xffffffffu, row_m, er & 31);
    const float c = __shfl_sync(0xffffffffu, row_c, er & 31);
    if (er < nrows && n0 + et < p.N) {
        const int64_t n = n0 + et;
        const int64_t o = p.out_mn ? (int64_t)m * p.ld_out + n : n * p.ld_out + m;
        p.out[o] = __fmul_rn(__int2float_rn(mine), c);
        if (p.acc) p.acc[o] = mine;
    }
}

template <int NT>
__global__ void __launch_bounds__(256, 2) grouped_kernel(const uint8_t* __restrict__ gtable, int use_smem)
{
    extern __shared__ __align__(16) uint8_t s_table[];
    const uint8_t* table = gtable;
    if (use_smem) {
        const int n16 = reinterpret_cast<const GroupedTable*>(gtable)->bytes >> 4;
        for (int i = threadIdx.x; i < n16; i += blockDim.x)
            reinterpret_cast<uint4*>(s_table)[i] = __ldg(reinterpret_cast<const uint4*>(gtable) + i);
        __syncthreads();
        table = s_table;
    }
    const GroupedTable* hdr = reinterpret_cast<const GroupedTable*>(table);
    const int64_t* cum = reinterpret_cast<const int64_t*>(table + sizeof(GroupedTable));
    const Problem* probs = reinterpret_cast<const Problem*>(table + hdr->prob_off);
    constexpr int RW4 = (NT == 1) ? 8 : 4, RW8 = (NT == 1) ? 4 : 2;
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int64_t total = hdr->total;
    int pi = 0;
    for (int64_t w = warp0; w < total; w += nwarps) {
        while (w >= cum[pi + 1]) ++pi;
        const Problem& p = probs[pi];
        const int64_t local = w - cum[pi];
        const int iP = (p.nP + RW4 - 1) / RW4, iF = (p.nF4 + RW4 - 1) / RW4, i8 = (p.n8 + RW8 - 1) / RW8;
        const int ipg = iP + iF + i8;
        int li;
        int64_t n0;
        if ((local >> 32) == 0) {                            // the usual case: 32-bit division
            const uint32_t q = (uint32_t)local / (uint32_t)ipg;
            li = (int)((uint32_t)local - q * (uint32_t)ipg);
            n0 = (int64_t)q * NT;
        } else {
            li = (int)(local % ipg);
            n0 = (local / ipg) * NT;
        }
        if (li < iP) {
            const int r0 = li * RW4;
            grouped_rows<kPoT4, NT, RW4>(p, r0, min(RW4, p.nP - r0), n0, lane);
        } else if (li < iP + iF) {
            const int r0 = (li - iP) * RW4;
            grouped_rows<kFixed4, NT, RW4>(p, p.nP + r0, min(RW4, p.nF4 - r0), n0, lane);
        } else {
            const int r0 = (li - iP - iF) * RW8;
            grouped_rows<kFixed8, NT, RW8>(p, p.nP + p.nF4 + r0, min(RW8, p.n8 - r0), n0, lane);
        }
    }
}

// One-token form, software-pipelined across work items.  The profile of the plain form above
// shows warps waiting on their weight loads four cycles out of eight: an item's loads are issued,
// waited for, consumed, and only then does the warp look at its next item.  Here a warp walks a
// flat sequence of steps -- a step is one 128-bit load per lane from each of the item's rows
// (8 rows of 4-bit codes or 4 rows of Fixed-8 codes: 128 bytes per lane, 4 KB per warp) -- and the
// loads of step i+1, which may belong to the next item or even the next layer, are issued before
// step i is expanded and multiplied, so every warp has weight bytes in flight all the time.
struct StreamItem {
    const Problem* p;
    const uint8_t* base;       // first row of the item
    uint32_t pitch;            // bytes per packed row
    int kind, nrows, nchunks;
    int row_m;                 // lane r: original index of row r
    float row_c;               // lane r: scale of row r
};

__device__ __forceinline__ bool stream_item(const uint8_t* table, int64_t w, int& pi, int lane, StreamItem& it)
{
    const GroupedTable* hdr = reinterpret_cast<const GroupedTable*>(table);
    if (w >= hdr->total) return false;
    const int64_t* cum = reinterpret_cast<const int64_t*>(table + sizeof(GroupedTable));
    const Problem* probs = reinterpret_cast<const Problem*>(table + hdr->prob_off);
    while (w >= cum[pi + 1]) ++pi;
    const Problem& p = probs[pi];
    const int li = (int)(w - cum[pi]);                       // one token: an item index inside the layer
    const int iP = (p.nP + 7) >> 3, iF = (p.nF4 + 7) >> 3;
    int pr0, rows_left;
    if (li < iP) { it.kind = kPoT4; pr0 = li * 8; rows_left = p.nP - pr0; }
    else if (li < iP + iF) { it.kind = kFixed4; pr0 = p.nP + (li - iP) * 8; rows_left = p.nP + p.nF4 - pr0; }
    else { it.kind = kFixed8; pr0 = p.nP + p.nF4 + (li - iP - iF) * 4; rows_left = p.M - pr0; }
    const int cap = (it.kind == kFixed8) ? 4 : 8;
    it.p = &p;
    it.nrows = rows_left < cap ? rows_left : cap;
    it.nchunks = p.Cp >> 5;
    if (it.kind == kFixed8) { it.pitch = (uint32_t)p.Kp; it.base = p.q8 + (size_t)(pr0 - p.nP - p.nF4) * it.pitch; }
    else { it.pitch = (uint32_t)p.Kp >> 1; it.base = p.q4 + (size_t)pr0 * it.pitch; }
    it.row_m = 0;
    it.row_c = 0.0f;
    if (lane < it.nrows) {
        it.row_m = __ldg(p.perm + pr0 + lane);
        it.row_c = __fmul_rn(__ldg(p.wstep + it.row_m), p.act_step);
    }
    return true;
}

// raw[r] = chunk `ch` of row r (4-bit kinds); raw[2r], raw[2r+1] = its two halves (Fixed-8).
__device__ __forceinline__ void stream_load(const StreamItem& it, int ch, uint4 (&raw)[8], uint4 (&act)[2])
{
    const bool live = ch < it.nchunks;
    // the token's 32 activation codes of this chunk travel with the weights (a ragged last chunk is
    // fetched bytewise at compute time instead)
    act[0] = act[1] = make_uint4(0, 0, 0, 0);
    if (live && (ch << 5) + 32 <= it.p->Cin) {
        const uint4* ap = reinterpret_cast<const uint4*>(it.p->act + (ch << 5));
        act[0] = __ldg(ap);
        act[1] = __ldg(ap + 1);
    }
    if (it.kind == kFixed8) {
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int rr = r < it.nrows ? r : it.nrows - 1;  // rows past the item's end repeat its last one
            const uint4* src = reinterpret_cast<const uint4*>(it.base + (size_t)rr * it.pitch + ((size_t)ch << 5));
            raw[2 * r] = live ? __ldcs(src) : make_uint4(0, 0, 0, 0);
            raw[2 * r + 1] = live ? __ldcs(src + 1) : make_uint4(0, 0, 0, 0);
        }
    } else {
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            const int rr = r < it.nrows ? r : it.nrows - 1;
            const uint4* src = reinterpret_cast<const uint4*>(it.base + (size_t)rr * it.pitch + ((size_t)ch << 4));
            raw[r] = live ? __ldcs(src) : make_uint4(0, 0, 0, 0);
        }
    }
}

__device__ __forceinline__ void stream_compute(const StreamItem& it, int ch, const uint4 (&raw)[8], const uint4 (&act)[2],
                                               int (&acc)[8])
{
    if (ch >= it.nchunks) return;
    const Problem& p = *it.p;
    const int kp = ch << 5;
    uint32_t a[8] = {act[0].x, act[0].y, act[0].z, act[0].w, act[1].x, act[1].y, act[1].z, act[1].w};
    if (kp + 32 > p.Cin) {
        const int8_t* ap = p.act + kp;                       // token 0
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            uint32_t v = 0;
#pragma unroll
            for (int bb = 0; bb < 4; ++bb)
                if (kp + q * 4 + bb < p.Cin) v |= (uint32_t)(uint8_t)ap[q * 4 + bb] << (8 * bb);
            a[q] = v;
        }
    }
    if (it.kind == kPoT4) {
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            const uint32_t c[4] = {raw[r].x, raw[r].y, raw[r].z, raw[r].w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {                    // eight codes at a time: few registers live
                uint32_t w0, w1;
                expand_pot_word(c[q], w0, w1);
                acc[r] = __dp4a((int)w1, (int)a[2 * q + 1], __dp4a((int)w0, (int)a[2 * q], acc[r]));
            }
        }
    } else if (it.kind == kFixed4) {
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            const uint32_t c[4] = {raw[r].x, raw[r].y, raw[r].z, raw[r].w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {                    // byte b: code b in the high, code 16 + b in the low nibble
                acc[r] = __dp4a((int)(c[q] & 0xF0F0F0F0u), (int)a[q], acc[r]);
                acc[r] = __dp4a((int)((c[q] << 4) & 0xF0F0F0F0u), (int)a[4 + q], acc[r]);
            }
        }
    } else {
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const uint32_t c[8] = {raw[2 * r].x, raw[2 * r].y, raw[2 * r].z, raw[2 * r].w,
                                   raw[2 * r + 1].x, raw[2 * r + 1].y, raw[2 * r + 1].z, raw[2 * r + 1].w};
#pragma unroll
            for (int q = 0; q < 8; ++q) acc[r] = __dp4a((int)c[q], (int)a[q], acc[r]);
        }
    }
}

__device__ __forceinline__ void stream_finish(const StreamItem& it, int lane, int (&acc)[8])
{
    const Problem& p = *it.p;
    int mine = 0;
#pragma unroll
    for (int r = 0; r < 8; ++r) {
        int v = __reduce_add_sync(0xffffffffu, acc[r]);
        if (it.kind == kFixed4) v >>= 4;                     // the Fixed-4 codes were expanded as 16 * value
        if (lane == r) mine = v;
        acc[r] = 0;
    }
    if (lane < it.nrows) {
        const int64_t o = p.out_mn ? (int64_t)it.row_m * p.ld_out : (int64_t)it.row_m;
        p.out[o] = __fmul_rn(__int2float_rn(mine), it.row_c);
        if (p.acc) p.acc[o] = mine;
    }
}

__global__ void __launch_bounds__(256, 2) grouped_stream_kernel(const uint8_t* __restrict__ gtable, int use_smem)
{
    extern __shared__ __align__(16) uint8_t s_table[];
    const uint8_t* table = gtable;
    if (use_smem) {
        const int n16 = reinterpret_cast<const GroupedTable*>(gtable)->bytes >> 4;
        for (int i = threadIdx.x; i < n16; i += blockDim.x)
            reinterpret_cast<uint4*>(s_table)[i] = __ldg(reinterpret_cast<const uint4*>(gtable) + i);
        __syncthreads();
        table = s_table;
    }
    const int lane = threadIdx.x & 31;
    int64_t w = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    StreamItem cur, nxt;
    int pi = 0;
    if (!stream_item(table, w, pi, lane, cur)) return;
    int ch = lane;
    uint4 rc[8], rn[8], ac[2], an[2];
    int acc[8];
#pragma unroll
    for (int r = 0; r < 8; ++r) acc[r] = 0;
    stream_load(cur, ch, rc, ac);
    for (;;) {
        const bool same = (ch - lane + 32) < cur.nchunks;    // warp-uniform: the item has another step
        bool more = true;
        if (same) {
            stream_load(cur, ch + 32, rn, an);
        } else {
            w += nwarps;
            more = stream_item(table, w, pi, lane, nxt);
            if (more) stream_load(nxt, lane, rn, an);
        }
        stream_compute(cur, ch, rc, ac, acc);
        if (same) {
            ch += 32;
        } else {
            stream_finish(cur, lane, acc);
            if (!more) break;
            cur = nxt;
            ch = lane;
        }
#pragma unroll
        for (int r = 0; r < 8; ++r) rc[r] = rn[r];
        ac[0] = an[0];
        ac[1] = an[1];
    }
}

size_t grouped_table_bytes(int count)
{
    size_t off = sizeof(GroupedTable) + sizeof(int64_t) * (size_t)(count + 1);
    off = (off + 15) / 16 * 16;
    return (off + sizeof(Problem) * (size_t)count + 15) / 16 * 16;
}

// Fills `h_table` (grouped_table_bytes(count) bytes) from the problems; returns the token group size.
int grouped_fill_table(const Problem* probs, int count, uint8_t* h_table)
{
    int64_t maxN = 1;
    for (int i = 0; i < count; ++i) maxN = probs[i].N > maxN ? probs[i].N : maxN;
    const int nt = (maxN == 1) ? 1 : kTok;
    const int rw4 = grouped_rw(kPoT4, nt), rw8 = grouped_rw(kFixed8, nt);
    memset(h_table, 0, grouped_table_bytes(count));
    GroupedTable* hdr = reinterpret_cast<GroupedTable*>(h_table);
    int64_t* cum = reinterpret_cast<int64_t*>(h_table + sizeof(GroupedTable));
    size_t off = sizeof(GroupedTable) + sizeof(int64_t) * (size_t)(count + 1);
    off = (off + 15) / 16 * 16;
    hdr->count = count;
    hdr->prob_off = (int32_t)off;
    hdr->bytes = (int32_t)grouped_table_bytes(count);
    cum[0] = 0;
    for (int i = 0; i < count; ++i) {
        const Problem& q = probs[i];
        const int64_t ipg = (q.nP + rw4 - 1) / rw4 + (q.nF4 + rw4 - 1) / rw4 + (q.n8 + rw8 - 1) / rw8;
        cum[i + 1] = cum[i] + ipg * ((q.N + nt - 1) / nt);
    }
    hdr->total = cum[count];
    memcpy(h_table + off, probs, sizeof(Problem) * (size_t)count);
    return nt;
}

cudaError_t launch_grouped(const uint8_t* d_table, size_t table_bytes, int64_t total, int nt, cudaStream_t st)
{
    int64_t blocks = (total + 7) / 8;
    if (blocks > (int64_t)sm_count() * 2) blocks = (int64_t)sm_count() * 2;                  // one resident wave: two blocks of 128-register threads per SM
    if (blocks < 1) blocks = 1;
    const int use_smem = table_bytes <= (size_t)kGroupedSmemMax;
    const size_t smem = use_smem ? table_bytes : 0;
    static bool attr_done[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_done[dev]) {
        cudaError_t e = cudaFuncSetAttribute(grouped_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kGroupedSmemMax);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(grouped_kernel<kTok>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGroupedSmemMax);
        if (e != cudaSuccess) return e;
        attr_done[dev] = true;
    }
    if (nt == 1) grouped_stream_kernel<<<(unsigned)blocks, 256, smem, st>>>(d_table, use_smem);
    else grouped_kernel<kTok><<<(unsigned)blocks, 256, smem, st>>>(d_table, use_smem);
    return cudaGetLastError();
}

}  // namespace rmsmp
