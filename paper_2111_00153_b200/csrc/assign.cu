// Row assignment on the device (Section 3.1: lower variance -> PoT; Section 3.3: ratio A:B:C; Algorithm 1's
// assignment block) and the packed buffer's metadata built from it, so that a layer can be quantized and
// packed from nothing but its fp32 weights and the ratio.
//
//   row_stats_kernel   per row: population variance in double by two plain passes in reduction order (the
//                      definition's order of additions, so that the ranking agrees with it bit for bit) and
//                      max |w|.  32 rows per warp-sized tile: the tile is read coalesced and walked row-wise
//                      from shared memory.
//   rank_kernel        rank of every row under the key (variance, row index): the number of rows that come
//                      before it.  M^2 / 2 comparisons, tiled through shared memory.
//   build_meta_kernel  one block: the kind of every row from its rank (the n8 highest ranks Fixed-8, the nP
//                      lowest PoT-4, the rest Fixed-4), the stable grouping by prefix sums over the rows in
//                      original order, and every metadata section of the packed buffer.
#include "common.cuh"

namespace rmsmp {

namespace {

constexpr int kStatRows = 32;

__global__ void __launch_bounds__(256) row_stats_kernel(const float* __restrict__ W, int M, int K, double* __restrict__ var,
                                                        float* __restrict__ amax)
{
    // 8 warps: each loads 4 rows x 32 columns of a 32 x 32 tile; thread r < 32 then walks row r of the tile
    __shared__ float tile[kStatRows][33];
    const int row0 = blockIdx.x * kStatRows;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int my_row = row0 + threadIdx.x;
    double sum = 0.0;
    float mx = 0.0f;
    for (int pass = 0; pass < 2; ++pass) {
        const double mean = (pass == 1) ? sum / (double)K : 0.0;
        double ss = 0.0;
        for (int k0 = 0; k0 < K; k0 += 32) {
            __syncthreads();
            for (int r = warp; r < kStatRows; r += 8) {
                const int row = row0 + r, k = k0 + lane;
                tile[r][lane] = (row < M && k < K) ? W[(size_t)row * K + k] : 0.0f;
            }
            __syncthreads();
            if (threadIdx.x < kStatRows && my_row < M) {
                const int kn = min(32, K - k0);
                for (int j = 0; j < kn; ++j) {
                    const float w = tile[threadIdx.x][j];
                    if (pass == 0) {
                        sum = __dadd_rn(sum, (double)w);
                        mx = fmaxf(mx, fabsf(w));
                    } else {
                        const double d = __dsub_rn((double)w, mean);
                        ss = __dadd_rn(ss, __dmul_rn(d, d));
                    }
                }
            }
        }
        if (pass == 1 && threadIdx.x < kStatRows && my_row < M) {
            var[my_row] = ss / (double)K;
            amax[my_row] = (mx == 0.0f) ? 1.0f : mx;
        }
    }
}

__global__ void __launch_bounds__(256) rank_kernel(const double* __restrict__ var, int M, int32_t* __restrict__ rank)
{
    __shared__ double s_var[256];
    const int r = blockIdx.x * 256 + threadIdx.x;
    const double mine = (r < M) ? var[r] : 0.0;
    int before = 0;
    for (int j0 = 0; j0 < M; j0 += 256) {
        __syncthreads();
        s_var[threadIdx.x] = (j0 + threadIdx.x < M) ? var[j0 + threadIdx.x] : 0.0;
        __syncthreads();
        const int jn = min(256, M - j0);
        for (int j = 0; j < jn; ++j) {
            const double v = s_var[j];
            before += (v < mine || (v == mine && j0 + j < r)) ? 1 : 0;
        }
    }
    if (r < M) rank[r] = before;
}

struct MetaArgs {
    uint8_t* blob;
    const int32_t* rank;
    const float* alpha;       // per row: the caller's, or the max |w| found by row_stats_kernel
    uint8_t* scheme_out;      // optional
    uint8_t* bits_out;        // optional
    uint64_t off_perm, off_slot, off_wstep, off_alpha, off_kind, off_blocks;
    int M, Cin, kh, kw, Cp, Kp, nP, nF4, n8, nblocks, pot_mode;
};

__global__ void __launch_bounds__(1024, 1) build_meta_kernel(MetaArgs a)
{
    __shared__ int s_cnt[3][1024];      // rows of each kind in this thread's chunk of rows, then exclusive prefix
    const int t = threadIdx.x, nt = blockDim.x;
    const int per = (a.M + nt - 1) / nt;                  // consecutive rows per thread: the grouping stays stable
    const int r0 = t * per, r1 = min(a.M, r0 + per);
    auto kind_of = [&](int r) -> int {
        const int rk = a.rank[r];
        return rk < a.nP ? kPoT4 : (rk < a.M - a.n8 ? kFixed4 : kFixed8);
    };
    int c[3] = {0, 0, 0};
    for (int r = r0; r < r1; ++r) ++c[kind_of(r)];
    for (int k = 0; k < 3; ++k) s_cnt[k][t] = c[k];
    __syncthreads();
    if (t < 3) {                                          // three serial scans of 1024 entries: negligible
        int run = 0;
        for (int i = 0; i < nt; ++i) { const int v = s_cnt[t][i]; s_cnt[t][i] = run; run += v; }
    }
    __syncthreads();
    int32_t* perm = reinterpret_cast<int32_t*>(a.blob + a.off_perm);
    int32_t* slot = reinterpret_cast<int32_t*>(a.blob + a.off_slot);
    float* wstep = reinterpret_cast<float*>(a.blob + a.off_wstep);
    float* alpha = reinterpret_cast<float*>(a.blob + a.off_alpha);
    uint8_t* kind = a.blob + a.off_kind;
    int32_t* blocks = reinterpret_cast<int32_t*>(a.blob + a.off_blocks);
    const int base[3] = {0, a.nP, a.nP + a.nF4};
    int next[3] = {s_cnt[0][t], s_cnt[1][t], s_cnt[2][t]};       // position inside each group
    for (int r = r0; r < r1; ++r) {
        const int k = kind_of(r);
        const int p = base[k] + next[k];
        perm[p] = r;
        slot[r] = p;
        kind[r] = (uint8_t)k;
        const float al = a.alpha[r];
        alpha[r] = al;
        wstep[r] = __fdiv_rn(al, k == kPoT4 ? 64.0f : (k == kFixed4 ? 7.0f : 127.0f));
        if (a.scheme_out) a.scheme_out[r] = (k == kPoT4) ? RMSMP_SCHEME_POT : RMSMP_SCHEME_FIXED;
        if (a.bits_out) a.bits_out[r] = (k == kFixed8) ? 8 : 4;
        ++next[k];
    }
    __syncthreads();
    // block table: first position (inside its group) and count of each kind among the block's 128 rows
    for (int b = t; b < a.nblocks; b += nt) {
        int cnt[3] = {0, 0, 0}, first[3] = {0, 0, 0};
        const int rb = b * kBlockRows, re = min(a.M, rb + kBlockRows);
        for (int r = rb; r < re; ++r) {
            const int k = kind[r];
            if (cnt[k] == 0) first[k] = slot[r] - base[k];
            ++cnt[k];
        }
        int32_t* be = blocks + 8 * b;
        be[0] = first[0]; be[1] = cnt[0]; be[2] = first[1]; be[3] = cnt[1]; be[4] = first[2]; be[5] = cnt[2]; be[6] = 0; be[7] = 0;
    }
    if (t == 0) {
        BlobHeader* H = reinterpret_cast<BlobHeader*>(a.blob);
        H->magic = kLayerMagic; H->version = kBlobVersion;
        H->M = a.M; H->Cin = a.Cin; H->kh = a.kh; H->kw = a.kw; H->Cp = a.Cp; H->Kp = a.Kp;
        H->nP = a.nP; H->nF4 = a.nF4; H->n8 = a.n8; H->nblocks = a.nblocks; H->pot_mode = a.pot_mode;
        H->pad0[0] = H->pad0[1] = H->pad0[2] = 0;
        H->status = 0;
    }
}

}  // namespace

size_t assign_scratch_bytes(int M) { return ((size_t)M * (8 + 4 + 4) + 255) / 256 * 256; }

cudaError_t launch_assign_meta(const float* dW, const rmsmp_layer& L, const float* d_alpha, int pot_mode, uint8_t* blob,
                               void* d_scratch, uint8_t* d_scheme, uint8_t* d_bits, cudaStream_t st)
{
    const int M = L.M, K = L.Cin * L.kh * L.kw;
    double* var = static_cast<double*>(d_scratch);
    int32_t* rank = reinterpret_cast<int32_t*>(var + M);
    float* amax = reinterpret_cast<float*>(rank + M);
    row_stats_kernel<<<(M + kStatRows - 1) / kStatRows, 256, 0, st>>>(dW, M, K, var, amax);
    rank_kernel<<<(M + 255) / 256, 256, 0, st>>>(var, M, rank);
    MetaArgs a;
    a.blob = blob; a.rank = rank; a.alpha = d_alpha ? d_alpha : amax; a.scheme_out = d_scheme; a.bits_out = d_bits;
    a.off_perm = L.off_perm; a.off_slot = L.off_slot; a.off_wstep = L.off_wstep; a.off_alpha = L.off_alpha;
    a.off_kind = L.off_kind; a.off_blocks = L.off_blocks;
    a.M = M; a.Cin = L.Cin; a.kh = L.kh; a.kw = L.kw; a.Cp = L.Cp; a.Kp = L.Kp;
    a.nP = L.nP; a.nF4 = L.nF4; a.n8 = L.n8; a.nblocks = L.nblocks; a.pot_mode = pot_mode;
    build_meta_kernel<<<1, 1024, 0, st>>>(a);
    return cudaGetLastError();
}

}  // namespace rmsmp
