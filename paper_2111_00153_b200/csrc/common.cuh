// Internal declarations shared by the translation units of librmsmp (not part of the ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include "../../include/rmsmp.h"

namespace rmsmp {

constexpr uint32_t kLayerMagic = 0x524D5350u;   // "RMSP"
constexpr uint32_t kBlobVersion = 1u;
constexpr int kBlockRows = 128;                  // rows of one MMA tile = one entry of `blocks`
constexpr int kStatusOffset = 64;                // byte offset of the device status word

enum RowKind : int { kPoT4 = 0, kFixed4 = 1, kFixed8 = 2 };

// First 256 bytes of a packed buffer.
struct BlobHeader {
    uint32_t magic, version;
    int32_t M, Cin, kh, kw, Cp, Kp, nP, nF4, n8, nblocks, pot_mode;
    int32_t pad0[3];
    uint32_t status;          // byte 64
    uint32_t pad1[47];
};
static_assert(sizeof(BlobHeader) == 256, "header is 256 bytes");
static_assert(offsetof(BlobHeader, status) == kStatusOffset, "status word at byte 64");

// Everything a contraction kernel needs; passed by value.
struct Problem {
    // weights
    const uint8_t* blob;
    const int32_t* perm;      // packed position -> original row
    const int32_t* slot;      // original row -> packed position
    const float* wstep;       // by original row
    const uint8_t* kind;      // by original row
    const int32_t* blocks;    // [nblocks][8]
    const uint8_t* q4;        // [(nP+nF4)][Kp/2]
    const uint8_t* q8;        // [n8][Kp]
    const int8_t* wexp;       // [M][Kp] int8 values in original row order, or null (workspace variant)
    uint32_t* status;
    int M, Cin, kh, kw, Cp, Kp, nP, nF4, n8, nblocks, raw_stage_bytes;
    // activations: [B][H][W] pixels of `pix_pitch` bytes, Cin codes used in each
    const int8_t* act;
    int B, H, W, Ho, Wo, stride, pad;
    int64_t pix_pitch;
    int64_t N;                // B*Ho*Wo
    int act_nonneg;           // grouped tensor-core launch: every activation code is within 0..15
    // outputs
    float act_step;
    float* out;
    int32_t* acc;             // may be null
    int64_t ld_out;
    int out_mn;               // 0: y[n*ld+m], 1: y[m*ld+n]
    // re-quantizing epilogue (tensor path, workspace mode): when rq_codes is set the kernel writes
    // the NEXT layer's 4-bit activation codes of y, codes[n*ld_codes+m], instead of y itself
    int8_t* rq_codes;
    float rq_alpha;
    int rq_kind;
    int64_t ld_codes;
};

// Per-device host state.  A process may drive several GPUs; anything learnt from or set on a device
// (its SM count, a kernel's shared-memory attribute) is cached by the device's ordinal, never once
// per process.  device_ordinal() returns the current device, or -1 when it cannot be had or lies
// beyond the tables (kMaxDevices).
constexpr int kMaxDevices = 64;
int device_ordinal();
int sm_count();               // SMs of the current device (cached per ordinal)
// Calls cudaFuncSetAttribute(MaxDynamicSharedMemorySize) for `fn` once per device: `done` is the
// kernel's own table of kMaxDevices flags.  Returns false if the attribute could not be set.
bool ensure_smem_attr(const void* fn, int bytes, bool* done);

// Re-quantizing epilogue request (rmsmp_*_workspace_requant): the next layer's clip value, kind and code buffer.
struct Requant {
    float alpha;
    rmsmp_act_kind kind;
    int8_t* codes;
    int64_t ld;
};

// host side of the linear-layer calls, split so that a caller can validate before it queues anything
// (host_api.cu): all checks + the problem description; then the launch of the chosen variant
rmsmp_status gemm_prepare(const rmsmp_layer* L, const void* d_packed, const void* d_ws, bool use_ws,
                          const int8_t* d_act, int64_t N, int64_t ld_act, float act_step, float* d_out,
                          int64_t ld_out, rmsmp_out_layout out_layout, int32_t* d_acc, const Requant* rq,
                          Problem& p);
rmsmp_status dispatch_problem(Problem& p, rmsmp_variant variant, cudaStream_t st);

// kernels (each returns the CUDA launch error, cudaSuccess if fine)
cudaError_t launch_pack(const float* dW, int conv_oihw, const rmsmp_layer& L, int pot_mode,
                        uint8_t* blob, cudaStream_t st);
// depthwise convolution on the CUDA cores (depthwise.cu)
bool depthwise_supported(const Problem& p);
cudaError_t launch_depthwise(const Problem& p, cudaStream_t st);
// patch matrix of a few-channel convolution (gather.cu)
cudaError_t launch_im2col(const int8_t* act, int B, int H, int W, int C, int64_t pix_pitch, int kh, int kw, int stride, int pad,
                          int Ho, int Wo, int8_t* cols, int64_t ld_cols, cudaStream_t st);
// row assignment on the device + the packed buffer's metadata (assign.cu); scratch of assign_scratch_bytes(M)
size_t assign_scratch_bytes(int M);
cudaError_t launch_assign_meta(const float* dW, const rmsmp_layer& L, const float* d_alpha, int pot_mode, uint8_t* blob,
                               void* d_scratch, uint8_t* d_scheme, uint8_t* d_bits, cudaStream_t st);
// copies `bytes` from mapped pinned host memory (device view, 16-byte aligned) to device memory
cudaError_t launch_fetch_mapped(void* d_dst, const void* mapped_src, size_t bytes, cudaStream_t st);
cudaError_t launch_unpack(const rmsmp_layer& L, const uint8_t* blob, int8_t* values,
                          int32_t* perm, float* wstep, cudaStream_t st);
cudaError_t launch_expand(const rmsmp_layer& L, const uint8_t* blob, int8_t* wexp, cudaStream_t st);
cudaError_t launch_quantize_act(const float* x, size_t count, float alpha, int kind, int8_t* codes,
                                cudaStream_t st);
cudaError_t launch_simple(const Problem& p, cudaStream_t st);
cudaError_t launch_simt(const Problem& p, bool shiftadd, cudaStream_t st);
size_t grouped_table_bytes(int count);
int grouped_fill_table(const Problem* probs, int count, uint8_t* h_table);
cudaError_t launch_grouped(const uint8_t* d_table, size_t table_bytes, int64_t total, int nt, cudaStream_t st);
// grouped tensor-core launch (stream.cu): table size, per-problem support test, host-side table and
// launch geometry, launch
int64_t stream_items_of(int nP, int nF4, int n8);
int64_t stream_act_bytes(int nP, int act_nonneg, int64_t N, int Kp);
size_t stream_table_bytes(int count, int64_t nitems, int sms, int64_t act_bytes);
bool stream_supported(const Problem& p);
bool stream_build_table(const Problem* probs, int count, int sms, uint8_t* h_table, size_t table_bytes,
                        uint8_t* d_table, int* grid_out, uint32_t* smem_out, uint32_t* conv_grid_out);
cudaError_t launch_stream(const uint8_t* d_table, int grid, uint32_t smem_bytes, int count, uint32_t conv_grid_x, cudaStream_t st);
// returns false if the tensor variant cannot run this problem (alignment / shape)
bool tensor_supported(const Problem& p);
rmsmp_status launch_tensor(const Problem& p, cudaStream_t st);
// fills four CUtensorMap objects (see act_parity_split; only the first is used without the split) for
// activation boxes of bk channels x th output rows x tb images, swizzle width = bk bytes
bool encode_act_maps_4(const Problem& p, int bk, int th, int tb, void* maps4);
// two-CTA form of the workspace mode (tensor2.cu): false if it cannot, or should not, run this problem
bool pair_supported(const Problem& p);
rmsmp_status launch_pair(const Problem& p, cudaStream_t st);

// ---- activation boxes of the tensor-core kernels ----
// A stride-2 convolution reads, for one filter tap, every second pixel of every second input row.
// Asking the copy engine for that with element strides makes it fetch pixel by pixel (measured: an
// order of magnitude below its unit-stride rate).  Instead the input is seen as four sub-grids by
// row and column parity, each with its own tensor map of doubled global strides and unit element
// strides; the pixels one tap needs for a whole tile lie in ONE sub-grid and form a dense box
// there.  Out-of-range coordinates of a sub-grid read zeros, which is the padding, as before.
__host__ __device__ inline bool act_parity_split(const Problem& p)
{
    return p.stride == 2 && p.H >= 2 && p.W >= 2;
}
struct TapBox { int map, x, y; };      // tensor map index (row parity * 2 + column parity), box start
__host__ __device__ inline TapBox tap_box(const Problem& p, int h0, int ti, int tj)
{
    TapBox t;
    const int dy = ti - p.pad, dx = tj - p.pad;
    if (act_parity_split(p)) {
        const int py = dy & 1, px = dx & 1;            // two's complement: -1 & 1 == 1
        t.map = py * 2 + px;
        t.y = h0 + ((dy - py) >> 1);                   // dy - py is even; arithmetic shift
        t.x = (dx - px) >> 1;
    } else {
        t.map = 0;
        t.y = h0 * p.stride + dy;
        t.x = dx;
    }
    return t;
}

// ---- device helpers used by more than one kernel file ----

// Integer value of a PoT-4 nibble (sign<<3 | e): 0 or +-2^(e-1).
__device__ __forceinline__ int pot_value(int nib)
{
    int e = nib & 7;
    int v = e ? (1 << (e - 1)) : 0;
    return (nib & 8) ? -v : v;
}

// Value of code k' of packed row `row4` (4-bit storage), see the layout in rmsmp.h.
__device__ __forceinline__ int decode4(const uint8_t* row4, int kprime, int kind)
{
    int chunk = kprime >> 5, o = kprime & 31;
    if (kind == kPoT4) {
        int byte = row4[chunk * 16 + (o >> 1)];
        return pot_value((o & 1) ? (byte >> 4) : (byte & 15));
    }
    int byte = row4[chunk * 16 + (o & 15)];
    int nib = (o < 16) ? (byte >> 4) : (byte & 15);
    return (nib ^ 8) - 8;
}

}  // namespace rmsmp
