// Host side of the C ABI: validation, layer description, metadata upload, dispatch.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <mutex>
#include <vector>
#include "common.cuh"

using namespace rmsmp;

namespace {

inline uint64_t align_up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }

constexpr uint32_t kPlanMagicHost = 0x47504C4Eu;   // "GPLN": rmsmp_grouped_plan filled by rmsmp_gemm_grouped_prepare

inline int row_kind(int scheme, int bits)
{
    if (scheme == RMSMP_SCHEME_POT && bits == 4) return kPoT4;
    if (scheme == RMSMP_SCHEME_FIXED && bits == 4) return kFixed4;
    if (scheme == RMSMP_SCHEME_FIXED && bits == 8) return kFixed8;
    return -1;
}

bool layer_ok(const rmsmp_layer* L)
{
    return L && L->magic == kLayerMagic && L->M >= 1 && L->Cin >= 1 && L->kh >= 1 && L->kw >= 1 &&
           L->nP + L->nF4 + L->n8 == L->M && L->packed_bytes >= 256;
}

rmsmp_status check_arch()
{
    const int dev = device_ordinal();
    static int cached_major[kMaxDevices];
    static bool have[kMaxDevices];
    if (dev < 0) return RMSMP_ERR_CUDA;
    if (!have[dev]) {
        int major = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
            cudaGetLastError();
            return RMSMP_ERR_CUDA;
        }
        cached_major[dev] = major;
        have[dev] = true;
    }
    return cached_major[dev] == 10 ? RMSMP_OK : RMSMP_ERR_ARCH;
}

// Pinned host staging for the metadata upload of rmsmp_quantize_pack.  A copy from pageable memory
// makes the host wait for the stream; from pinned memory it is asynchronous.  The slot is mapped
// into the device's address space and a small kernel fetches it: between two kernels of a stream a
// copy-engine transfer of a few KB costs several microseconds more than a kernel does.  One small ring of
// slots per device, created on first use (host memory only; no device memory is ever allocated);
// an event per slot tells when its last copy has left.  If pinned memory cannot be had, or the
// metadata is larger than a slot, the pageable path is used.
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

constexpr size_t kStageSlotBytes = 64 * 1024;
constexpr int kStageSlots = 32;
struct StageRing {
    bool tried = false;
    uint8_t* base = nullptr;
    uint8_t* dev_base = nullptr;      // the same memory as the device sees it
    cudaEvent_t ev[kStageSlots];
    bool used[kStageSlots];
    int next = 0;
};
StageRing g_stage[kMaxDevices];
std::mutex g_stage_mutex;

// Copies `bytes` of metadata to the device through a pinned slot; false = caller uses the pageable path.
bool staged_upload(void* d_dst, const void* h_src, size_t bytes, cudaStream_t st)
{
    if (bytes > kStageSlotBytes) return false;
    const int dev = device_ordinal();
    if (dev < 0) return false;
    std::lock_guard<std::mutex> lock(g_stage_mutex);
    StageRing& r = g_stage[dev];
    if (!r.tried) {
        r.tried = true;
        void* ptr = nullptr;
        if (cudaHostAlloc(&ptr, kStageSlotBytes * kStageSlots, cudaHostAllocMapped) != cudaSuccess) {
            cudaGetLastError();
        } else {
            bool ok = true;
            for (int i = 0; i < kStageSlots; ++i) {
                r.used[i] = false;
                if (cudaEventCreateWithFlags(&r.ev[i], cudaEventDisableTiming) != cudaSuccess) { cudaGetLastError(); ok = false; break; }
            }
            void* dptr = nullptr;
            if (ok && cudaHostGetDevicePointer(&dptr, ptr, 0) != cudaSuccess) { cudaGetLastError(); dptr = nullptr; }
            if (ok) { r.base = static_cast<uint8_t*>(ptr); r.dev_base = static_cast<uint8_t*>(dptr); } else cudaFreeHost(ptr);
        }
    }
    if (!r.base) return false;
    const int slot = r.next;
    r.next = (r.next + 1) % kStageSlots;
    if (r.used[slot] && cudaEventSynchronize(r.ev[slot]) != cudaSuccess) { cudaGetLastError(); return false; }
    uint8_t* h = r.base + (size_t)slot * kStageSlotBytes;
    std::memcpy(h, h_src, bytes);
    const bool by_kernel = r.dev_base && aligned16(d_dst) &&
                           launch_fetch_mapped(d_dst, r.dev_base + (size_t)slot * kStageSlotBytes, bytes, st) == cudaSuccess;
    if (!by_kernel) {
        cudaGetLastError();
        if (cudaMemcpyAsync(d_dst, h, bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) { cudaGetLastError(); return false; }
    }
    if (cudaEventRecord(r.ev[slot], st) != cudaSuccess) { cudaGetLastError(); return false; }
    r.used[slot] = true;
    return true;
}

void fill_problem(Problem& p, const rmsmp_layer* L, const void* d_packed)
{
    const uint8_t* blob = static_cast<const uint8_t*>(d_packed);
    p.blob = blob;
    p.perm = reinterpret_cast<const int32_t*>(blob + L->off_perm);
    p.slot = reinterpret_cast<const int32_t*>(blob + L->off_slot);
    p.wstep = reinterpret_cast<const float*>(blob + L->off_wstep);
    p.kind = blob + L->off_kind;
    p.blocks = reinterpret_cast<const int32_t*>(blob + L->off_blocks);
    p.q4 = blob + L->off_q4;
    p.q8 = blob + L->off_q8;
    p.status = reinterpret_cast<uint32_t*>(const_cast<uint8_t*>(blob) + kStatusOffset);
    p.M = L->M; p.Cin = L->Cin; p.kh = L->kh; p.kw = L->kw; p.Cp = L->Cp; p.Kp = L->Kp;
    p.nP = L->nP; p.nF4 = L->nF4; p.n8 = L->n8; p.nblocks = L->nblocks;
    p.raw_stage_bytes = L->raw_stage_bytes;
    p.wexp = nullptr;
    p.rq_codes = nullptr; p.rq_alpha = 1.0f; p.rq_kind = 0; p.ld_codes = 0;
}

rmsmp_status dispatch(Problem& p, rmsmp_variant variant, cudaStream_t st)
{
    if (variant == RMSMP_VARIANT_AUTO) {
        if (p.N >= 32 && tensor_supported(p)) variant = RMSMP_VARIANT_TENSOR;
        else variant = RMSMP_VARIANT_SIMT;
    }
    cudaError_t e = cudaSuccess;
    switch (variant) {
        case RMSMP_VARIANT_TENSOR:
            if (!tensor_supported(p)) return RMSMP_ERR_VARIANT;
            return launch_tensor(p, st);
        case RMSMP_VARIANT_SIMT: e = launch_simt(p, false, st); break;
        case RMSMP_VARIANT_SHIFTADD: e = launch_simt(p, true, st); break;
        case RMSMP_VARIANT_SIMPLE: e = launch_simple(p, st); break;
        default: return RMSMP_ERR_VARIANT;
    }
    return e == cudaSuccess ? RMSMP_OK : RMSMP_ERR_CUDA;
}

}  // namespace

#include <nvtx3/nvToolsExt.h>

// A named NVTX range around every call that queues GPU work: a profiler's timeline shows which API call a
// kernel belongs to.  Without a tool attached the two calls return at once.
struct NvtxRange {
    explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
    ~NvtxRange() { nvtxRangePop(); }
    NvtxRange(const NvtxRange&) = delete;
    NvtxRange& operator=(const NvtxRange&) = delete;
};

namespace rmsmp {

int device_ordinal()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return -1; }
    return (dev >= 0 && dev < kMaxDevices) ? dev : -1;
}

int sm_count()
{
    static int cached[kMaxDevices];
    const int dev = device_ordinal();
    if (dev < 0) return 1;
    if (cached[dev] == 0) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) cudaGetLastError();
        cached[dev] = v > 0 ? v : 1;
    }
    return cached[dev];
}

bool ensure_smem_attr(const void* fn, int bytes, bool* done)
{
    const int dev = device_ordinal();
    if (dev < 0) return false;
    if (!done[dev]) {
        if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) {
            cudaGetLastError();
            return false;
        }
        done[dev] = true;
    }
    return true;
}

}  // namespace rmsmp

extern "C" {

const char* rmsmp_status_string(rmsmp_status s)
{
    switch (s) {
        case RMSMP_OK: return "ok";
        case RMSMP_ERR_NULL: return "null pointer";
        case RMSMP_ERR_SHAPE: return "bad shape";
        case RMSMP_ERR_SCHEME: return "scheme/bits not in {PoT-4, Fixed-4, Fixed-8}";
        case RMSMP_ERR_SCALE: return "clip value not finite and positive";
        case RMSMP_ERR_ALIGN: return "pointer or leading dimension not 16-byte aligned";
        case RMSMP_ERR_BUFFER_TOO_SMALL: return "packed buffer too small";
        case RMSMP_ERR_ARCH: return "device is not sm_100";
        case RMSMP_ERR_CUDA: return "CUDA call failed";
        case RMSMP_ERR_TIMEOUT: return "bounded device wait ran out";
        case RMSMP_ERR_BAD_LAYER: return "layer descriptor not initialised";
        case RMSMP_ERR_VARIANT: return "kernel variant cannot run this problem";
    }
    return "unknown status";
}

rmsmp_status rmsmp_assign_rows(const float* h_W, int M, int K, int A, int B, int C,
                               uint8_t* h_scheme, uint8_t* h_bits)
{
    if (!h_W || !h_scheme || !h_bits) return RMSMP_ERR_NULL;
    if (M < 1 || K < 1 || A < 0 || B < 0 || C < 0 || A + B + C != 100) return RMSMP_ERR_SHAPE;
    // population variance per row, double, two plain passes
    std::vector<std::pair<double, int>> rank((size_t)M);
    for (int r = 0; r < M; ++r) {
        const float* w = h_W + (size_t)r * K;
        double sum = 0.0;
        for (int k = 0; k < K; ++k) sum += (double)w[k];
        const double mean = sum / (double)K;
        double ss = 0.0;
        for (int k = 0; k < K; ++k) {
            const double d = (double)w[k] - mean;
            ss += d * d;
        }
        rank[(size_t)r] = {ss / (double)K, r};
    }
    std::sort(rank.begin(), rank.end());   // (variance, row) ascending
    int n8 = (int)std::floor((double)M * C / 100.0 + 0.5);
    n8 = std::min(n8, M);
    int nP = (int)std::floor((double)M * A / 100.0 + 0.5);
    nP = std::min(nP, M - n8);
    for (int i = 0; i < M; ++i) {
        const int r = rank[(size_t)i].second;
        if (i < nP) { h_scheme[r] = RMSMP_SCHEME_POT; h_bits[r] = 4; }
        else if (i < M - n8) { h_scheme[r] = RMSMP_SCHEME_FIXED; h_bits[r] = 4; }
        else { h_scheme[r] = RMSMP_SCHEME_FIXED; h_bits[r] = 8; }
    }
    return RMSMP_OK;
}

// Shape checks, padded sizes and section offsets of a layer with cnt[] rows per kind.
static rmsmp_status layer_layout(rmsmp_layer* L, int M, int Cin, int kh, int kw, const int cnt[3])
{
    if (M < 1 || M > (1 << 20) || Cin < 1 || kh < 1 || kw < 1 || kh > 16 || kw > 16)
        return RMSMP_ERR_SHAPE;
    if ((int64_t)Cin * kh * kw > 1000000) return RMSMP_ERR_SHAPE;
    std::memset(L, 0, sizeof(*L));
    L->magic = kLayerMagic;
    L->M = M; L->Cin = Cin; L->kh = kh; L->kw = kw;
    L->Cp = (Cin + 31) / 32 * 32;
    L->Kp = (int32_t)align_up((uint64_t)kh * kw * L->Cp, 128);
    if (kh * kw > 1 && L->Kp > 196608) return RMSMP_ERR_SHAPE;   // one shared-memory segment in the pack kernel
    L->nP = cnt[0]; L->nF4 = cnt[1]; L->n8 = cnt[2];
    L->nblocks = (M + kBlockRows - 1) / kBlockRows;
    uint64_t off = 256;
    L->off_perm = off;   off = align_up(off + 4ull * M, 256);
    L->off_slot = off;   off = align_up(off + 4ull * M, 256);
    L->off_wstep = off;  off = align_up(off + 4ull * M, 256);
    L->off_alpha = off;  off = align_up(off + 4ull * M, 256);
    L->off_kind = off;   off = align_up(off + 1ull * M, 256);
    L->off_blocks = off; off = align_up(off + 32ull * L->nblocks, 256);
    L->off_q4 = off;     off = align_up(off + (uint64_t)(cnt[0] + cnt[1]) * (L->Kp / 2), 256);
    L->off_q8 = off;     off = align_up(off + (uint64_t)cnt[2] * L->Kp, 256);
    L->packed_bytes = off;
    return RMSMP_OK;
}

rmsmp_status rmsmp_layer_init(rmsmp_layer* L, int M, int Cin, int kh, int kw,
                              const uint8_t* h_scheme, const uint8_t* h_bits)
{
    if (!L || !h_scheme || !h_bits) return RMSMP_ERR_NULL;
    if (M < 1 || M > (1 << 20)) return RMSMP_ERR_SHAPE;
    int cnt[3] = {0, 0, 0};
    for (int r = 0; r < M; ++r) {
        const int k = row_kind(h_scheme[r], h_bits[r]);
        if (k < 0) return RMSMP_ERR_SCHEME;
        ++cnt[k];
    }
    rmsmp_status s = layer_layout(L, M, Cin, kh, kw, cnt);
    if (s != RMSMP_OK) return s;
    // bytes one k-block of one block's packed rows takes when fetched group by group in 16-row boxes
    int raw_max = 0;
    for (int b0 = 0; b0 < M; b0 += kBlockRows) {
        int c[3] = {0, 0, 0};
        for (int r = b0; r < M && r < b0 + kBlockRows; ++r) ++c[row_kind(h_scheme[r], h_bits[r])];
        const int bytes = ((c[0] + 15) / 16 * 16 + (c[1] + 15) / 16 * 16) * 64 + (c[2] + 15) / 16 * 16 * 128;
        raw_max = std::max(raw_max, bytes);
    }
    L->raw_stage_bytes = raw_max;
    return RMSMP_OK;
}

static void ratio_counts(int M, int A, int C, int cnt[3])
{
    int n8 = (int)std::floor((double)M * C / 100.0 + 0.5);
    n8 = std::min(n8, M);
    int nP = (int)std::floor((double)M * A / 100.0 + 0.5);
    nP = std::min(nP, M - n8);
    cnt[0] = nP; cnt[1] = M - nP - n8; cnt[2] = n8;
}

rmsmp_status rmsmp_layer_init_ratio(rmsmp_layer* L, int M, int Cin, int kh, int kw, int A, int B, int C)
{
    if (!L) return RMSMP_ERR_NULL;
    if (M < 1 || M > 65536 || A < 0 || B < 0 || C < 0 || A + B + C != 100) return RMSMP_ERR_SHAPE;
    int cnt[3];
    ratio_counts(M, A, C, cnt);
    rmsmp_status s = layer_layout(L, M, Cin, kh, kw, cnt);
    if (s != RMSMP_OK) return s;
    // which rows share a 128-row block is not known before the weights are ranked: the most a block can need
    auto up16 = [](int n) { return (n + 15) / 16 * 16; };
    L->raw_stage_bytes = (up16(std::min(kBlockRows, cnt[0])) + up16(std::min(kBlockRows, cnt[1]))) * 64 +
                         up16(std::min(kBlockRows, cnt[2])) * 128;
    return RMSMP_OK;
}

rmsmp_status rmsmp_assign_scratch_bytes(int M, size_t* bytes)
{
    if (!bytes) return RMSMP_ERR_NULL;
    if (M < 1 || M > 65536) return RMSMP_ERR_SHAPE;
    *bytes = assign_scratch_bytes(M);
    return RMSMP_OK;
}

rmsmp_status rmsmp_assign_quantize_pack(const float* d_W, rmsmp_w_layout w_layout, const rmsmp_layer* L, int A, int B,
                                        int C, const float* d_alpha, rmsmp_pot_mode pot_mode, void* d_packed,
                                        size_t packed_bytes, void* d_scratch, size_t scratch_bytes, uint8_t* d_scheme,
                                        uint8_t* d_bits, void* stream)
{
    NvtxRange nvtx_range("rmsmp_assign_quantize_pack");
    if (!d_W || !L || !d_packed || !d_scratch) return RMSMP_ERR_NULL;
    if (!layer_ok(L)) return RMSMP_ERR_BAD_LAYER;
    if (L->M > 65536 || A < 0 || B < 0 || C < 0 || A + B + C != 100) return RMSMP_ERR_SHAPE;
    if (w_layout != RMSMP_W_LINEAR && w_layout != RMSMP_W_CONV_OIHW) return RMSMP_ERR_SHAPE;
    if (w_layout == RMSMP_W_LINEAR && (L->kh != 1 || L->kw != 1)) return RMSMP_ERR_SHAPE;
    if (pot_mode != RMSMP_POT_NEAREST && pot_mode != RMSMP_POT_LOG2) return RMSMP_ERR_SCHEME;
    int cnt[3];
    ratio_counts(L->M, A, C, cnt);
    if (cnt[0] != L->nP || cnt[1] != L->nF4 || cnt[2] != L->n8) return RMSMP_ERR_SCHEME;   // descriptor of another ratio
    if (packed_bytes < L->packed_bytes || scratch_bytes < assign_scratch_bytes(L->M)) return RMSMP_ERR_BUFFER_TOO_SMALL;
    if (!aligned16(d_W) || (reinterpret_cast<uintptr_t>(d_packed) & 255) != 0 || !aligned16(d_scratch)) return RMSMP_ERR_ALIGN;
    rmsmp_status a = check_arch();
    if (a != RMSMP_OK) return a;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (launch_assign_meta(d_W, *L, d_alpha, pot_mode, static_cast<uint8_t*>(d_packed), d_scratch, d_scheme, d_bits, st) != cudaSuccess ||
        launch_pack(d_W, w_layout == RMSMP_W_CONV_OIHW, *L, pot_mode, static_cast<uint8_t*>(d_packed), st) != cudaSuccess) {
        cudaGetLastError();
        return RMSMP_ERR_CUDA;
    }
    return RMSMP_OK;
}

rmsmp_status rmsmp_quantize_pack(const float* d_W, rmsmp_w_layout w_layout, const rmsmp_layer* L,
                                 const uint8_t* h_scheme, const uint8_t* h_bits,
                                 const float* h_alpha, rmsmp_pot_mode pot_mode, void* d_packed,
                                 size_t packed_bytes, void* stream)
{
    NvtxRange nvtx_range("rmsmp_quantize_pack");
    if (!d_W || !L || !h_scheme || !h_bits || !h_alpha || !d_packed) return RMSMP_ERR_NULL;
    if (!layer_ok(L)) return RMSMP_ERR_BAD_LAYER;
    if (w_layout != RMSMP_W_LINEAR && w_layout != RMSMP_W_CONV_OIHW) return RMSMP_ERR_SHAPE;
    if (w_layout == RMSMP_W_LINEAR && (L->kh != 1 || L->kw != 1)) return RMSMP_ERR_SHAPE;
    if (pot_mode != RMSMP_POT_NEAREST && pot_mode != RMSMP_POT_LOG2) return RMSMP_ERR_SCHEME;
    if (packed_bytes < L->packed_bytes) return RMSMP_ERR_BUFFER_TOO_SMALL;
    if (!aligned16(d_W) || (reinterpret_cast<uintptr_t>(d_packed) & 255) != 0) return RMSMP_ERR_ALIGN;
    const int M = L->M;
    int cnt[3] = {0, 0, 0};
    for (int r = 0; r < M; ++r) {
        const int k = row_kind(h_scheme[r], h_bits[r]);
        if (k < 0) return RMSMP_ERR_SCHEME;
        ++cnt[k];
        if (!(h_alpha[r] > 0.0f) || !std::isfinite(h_alpha[r])) return RMSMP_ERR_SCALE;
    }
    if (cnt[0] != L->nP || cnt[1] != L->nF4 || cnt[2] != L->n8) return RMSMP_ERR_SCHEME;
    rmsmp_status a = check_arch();
    if (a != RMSMP_OK) return a;

    // metadata: everything before the code regions, built on the host and sent in one copy
    std::vector<uint8_t> meta((size_t)L->off_q4, 0);
    BlobHeader* H = reinterpret_cast<BlobHeader*>(meta.data());
    H->magic = kLayerMagic; H->version = kBlobVersion;
    H->M = M; H->Cin = L->Cin; H->kh = L->kh; H->kw = L->kw; H->Cp = L->Cp; H->Kp = L->Kp;
    H->nP = L->nP; H->nF4 = L->nF4; H->n8 = L->n8; H->nblocks = L->nblocks; H->pot_mode = pot_mode;
    H->status = 0;
    int32_t* perm = reinterpret_cast<int32_t*>(meta.data() + L->off_perm);
    int32_t* slot = reinterpret_cast<int32_t*>(meta.data() + L->off_slot);
    float* wstep = reinterpret_cast<float*>(meta.data() + L->off_wstep);
    float* alpha = reinterpret_cast<float*>(meta.data() + L->off_alpha);
    uint8_t* kind = meta.data() + L->off_kind;
    int32_t* blocks = reinterpret_cast<int32_t*>(meta.data() + L->off_blocks);
    int next[3] = {0, cnt[0], cnt[0] + cnt[1]};          // stable grouping
    for (int r = 0; r < M; ++r) {
        const int k = row_kind(h_scheme[r], h_bits[r]);
        const int blk = r / kBlockRows;
        int32_t* be = blocks + 8 * blk;
        const int rel = next[k] - (k == 0 ? 0 : (k == 1 ? cnt[0] : cnt[0] + cnt[1]));
        if (be[2 * k + 1] == 0) be[2 * k] = rel;
        be[2 * k + 1] += 1;
        perm[next[k]] = r;
        slot[r] = next[k];
        ++next[k];
        kind[r] = (uint8_t)k;
        alpha[r] = h_alpha[r];
        const float q = (k == kPoT4) ? 64.0f : (k == kFixed4 ? 7.0f : 127.0f);
        wstep[r] = h_alpha[r] / q;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!staged_upload(d_packed, meta.data(), meta.size(), st) &&
        cudaMemcpyAsync(d_packed, meta.data(), meta.size(), cudaMemcpyHostToDevice, st) != cudaSuccess) {
        cudaGetLastError();
        return RMSMP_ERR_CUDA;
    }
    if (launch_pack(d_W, w_layout == RMSMP_W_CONV_OIHW, *L, pot_mode, static_cast<uint8_t*>(d_packed), st) !=
        cudaSuccess) {
        cudaGetLastError();
        return RMSMP_ERR_CUDA;
    }
    return RMSMP_OK;
}

rmsmp_status rmsmp_unpack_codes(const rmsmp_layer* L, const void* d_packed, int8_t* d_values,
                                int32_t* d_perm, float* d_wstep, void* stream)
{
    NvtxRange nvtx_range("rmsmp_unpack_codes");
    if (!L || !d_packed || !d_values) return RMSMP_ERR_NULL;
    if (!layer_ok(L)) return RMSMP_ERR_BAD_LAYER;
    rmsmp_status a = check_arch();
    if (a != RMSMP_OK) return a;
    if (launch_unpack(*L, static_cast<const uint8_t*>(d_packed), d_values, d_perm, d_wstep,
                      static_cast<cudaStream_t>(stream)) != cudaSuccess) {
        cudaGetLastError();
        return RMSMP_ERR_CUDA;
    }
    return RMSMP_OK;
}

rmsmp_status rmsmp_quantize_act(const float* d_X, size_t count, float alpha_a, rmsmp_act_kind kind,
                                int8_t* d_codes, float* h_act_step, void* stream)
{
    NvtxRange nvtx_range("rmsmp_quantize_act");
    if (!d_X || !d_codes) return RMSMP_ERR_NULL;
    if (count < 1) return RMSMP_ERR_SHAPE;
    if (kind != RMSMP_ACT_U4 && kind != RMSMP_ACT_S4) return RMSMP_ERR_SCHEME;
    if (!(alpha_a > 0.0f) || !std::isfinite(alpha_a)) return RMSMP_ERR_SCALE;
    if (h_act_step) *h_act_step = alpha_a / (kind == RMSMP_ACT_U4 ? 15.0f : 7.0f);
    rmsmp_status a = check_arch();
    if (a != RMSMP_OK) return a;
    if (launch_quantize_act(d_X, count, alpha_a, kind, d_codes, static_cast<cudaStream_t>(stream)) !=
        cudaSuccess) {
        cudaGetLastError();
        return RMSMP_ERR_CUDA;
    }
    return RMSMP_OK;
}

static rmsmp_status requant_check(const Requant* rq, float* h_next_step)
{
    if (!rq->codes) return RMSMP_ERR_NULL;
    if (rq->kind != RMSMP_ACT_U4 && rq->kind != RMSMP_ACT_S4) return RMSMP_ERR_SCHEME;
    if (!(rq->alpha > 0.0f) || !std::isfinite(rq->alpha)) return RMSMP_ERR_SCALE;
    if (h_next_step) *h_next_step = rq->alpha / (rq->kind == RMSMP_ACT_U4 ? 15.0f : 7.0f);
    return RMSMP_OK;
}

}  // extern "C"

namespace rmsmp {

// Every host-side check of a linear-layer call, and the kernel's problem description.  Nothing is
// launched here, so a caller can validate first and queue work only for calls that will go through.
rmsmp_status gemm_prepare(const rmsmp_layer* L, const void* d_packed, const void* d_ws, bool use_ws,
                          const int8_t* d_act, int64_t N, int64_t ld_act, float act_step, float* d_out,
                          int64_t ld_out, rmsmp_out_layout out_layout, int32_t* d_acc, const Requant* rq,
                          Problem& p)
{
    if (!L || !d_packed || !d_act || (!d_out && !rq) || (use_ws && !d_ws)) return RMSMP_ERR_NULL;
    if (!layer_ok(L)) return RMSMP_ERR_BAD_LAYER;
    if (L->kh != 1 || L->kw != 1) return RMSMP_ERR_SHAPE;
    if (N < 1 || N > (int64_t)1 << 31 || ld_act < L->Cin) return RMSMP_ERR_SHAPE;
    if (out_layout != RMSMP_OUT_NM && out_layout != RMSMP_OUT_MN) return RMSMP_ERR_SHAPE;
    if (!rq && ld_out < (out_layout == RMSMP_OUT_NM ? (int64_t)L->M : N)) return RMSMP_ERR_SHAPE;
    if (rq && rq->ld < L->M) return RMSMP_ERR_SHAPE;
    if (!std::isfinite(act_step)) return RMSMP_ERR_SCALE;
    if (!aligned16(d_act) || (!rq && !aligned16(d_out)) || (d_acc && !aligned16(d_acc)) || (ld_act & 15) ||
        (reinterpret_cast<uintptr_t>(d_packed) & 255))
        return RMSMP_ERR_ALIGN;
    if (use_ws && !aligned16(d_ws)) return RMSMP_ERR_ALIGN;
    rmsmp_status a = check_arch();
    if (a != RMSMP_OK) return a;
    fill_problem(p, L, d_packed);
    p.act = d_act;
    p.B = (int)std::min<int64_t>(N, 0x7fffffff); p.H = 1; p.W = 1; p.Ho = 1; p.Wo = 1; p.stride = 1; p.pad = 0;
    p.pix_pitch = ld_act; p.N = N;
    p.act_step = act_step; p.out = d_out; p.acc = d_acc; p.ld_out = ld_out;
    p.out_mn = (out_layout == RMSMP_OUT_MN);
    if (rq) { p.rq_codes = rq->codes; p.rq_alpha = rq->alpha; p.rq_kind = rq->kind; p.ld_codes = rq->ld; }
    if (use_ws) p.wexp = static_cast<const int8_t*>(d_ws);
    return RMSMP_OK;
}

rmsmp_status dispatch_problem(Problem& p, rmsmp_variant variant, cudaStream_t st) { return dispatch(p, variant, st); }

}  // namespace rmsmp

static rmsmp_status gemm_impl(const rmsmp_layer* L, const void* d_packed, const void* d_ws, bool use_ws,
                              const int8_t* d_act, int64_t N, int64_t ld_act, float act_step, float* d_out,
                              int64_t ld_out, rmsmp_out_layout out_layout, int32_t* d_acc,
                              rmsmp_variant variant, void* stream, const Requant* rq = nullptr)
{
    Problem p;
    rmsmp_status s = gemm_prepare(L, d_packed, d_ws, use_ws, d_act, N, ld_act, act_step, d_out, ld_out, out_layout,
                                  d_acc, rq, p);
    if (s != RMSMP_OK) return s;
    return dispatch(p, variant, static_cast<cudaStream_t>(stream));
}

extern "C" {

rmsmp_status rmsmp_grouped_table_bytes(int count, size_t* bytes)
{
    if (!bytes) return RMSMP_ERR_NULL;
    if (count < 1 || count > 65536) return RMSMP_ERR_SHAPE;
    *bytes = (grouped_table_bytes(count) + 255) / 256 * 256;
    return RMSMP_OK;
}

// Host checks of a grouped call's items and their problem descriptions (nothing is launched).
static rmsmp_status grouped_problems(const rmsmp_gemm_item* h_items, int count, rmsmp_out_layout out_layout,
                                     std::vector<Problem>& probs)
{
    if (!h_items) return RMSMP_ERR_NULL;
    if (count < 1 || count > 65536) return RMSMP_ERR_SHAPE;
    if (out_layout != RMSMP_OUT_NM && out_layout != RMSMP_OUT_MN) return RMSMP_ERR_SHAPE;
    probs.resize((size_t)count);
    for (int i = 0; i < count; ++i) {
        const rmsmp_gemm_item& it = h_items[i];
        const rmsmp_layer* L = it.layer;
        if (!L || !it.d_packed || !it.d_act || !it.d_out) return RMSMP_ERR_NULL;
        if (!layer_ok(L)) return RMSMP_ERR_BAD_LAYER;
        if (L->kh != 1 || L->kw != 1) return RMSMP_ERR_SHAPE;
        if (it.N < 1 || it.N > (int64_t)1 << 31 || it.ld_act < L->Cin) return RMSMP_ERR_SHAPE;
        if (it.ld_out < (out_layout == RMSMP_OUT_NM ? (int64_t)L->M : it.N)) return RMSMP_ERR_SHAPE;
        if (!std::isfinite(it.act_step)) return RMSMP_ERR_SCALE;
        if (!aligned16(it.d_act) || !aligned16(it.d_out) || (it.d_acc && !aligned16(it.d_acc)) || (it.ld_act & 15) ||
            (reinterpret_cast<uintptr_t>(it.d_packed) & 255))
            return RMSMP_ERR_ALIGN;
        Problem& p = probs[(size_t)i];
        fill_problem(p, L, it.d_packed);
        p.act = it.d_act;
        p.B = (int)std::min<int64_t>(it.N, 0x7fffffff); p.H = 1; p.W = 1; p.Ho = 1; p.Wo = 1; p.stride = 1; p.pad = 0;
        p.pix_pitch = it.ld_act; p.N = it.N;
        p.act_step = it.act_step; p.out = it.d_out; p.acc = it.d_acc; p.ld_out = it.ld_out;
        p.out_mn = (out_layout == RMSMP_OUT_MN);
        p.act_nonneg = it.act_nonneg != 0;
    }
    return RMSMP_OK;
}

rmsmp_status rmsmp_gemm_grouped(const rmsmp_gemm_item* h_items, int count, rmsmp_out_layout out_layout,
                                void* d_table, size_t table_bytes, void* stream)
{
    NvtxRange nvtx_range("rmsmp_gemm_grouped");
    if (!d_table) return RMSMP_ERR_NULL;
    std::vector<Problem> probs;
    rmsmp_status s = grouped_problems(h_items, count, out_layout, probs);
    if (s != RMSMP_OK) return s;
    if (table_bytes < grouped_table_bytes(count)) return RMSMP_ERR_BUFFER_TOO_SMALL;
    if (!aligned16(d_table)) return RMSMP_ERR_ALIGN;
    rmsmp_status a = check_arch();
    if (a != RMSMP_OK) return a;
    std::vector<uint8_t> table(grouped_table_bytes(count));
    const int nt = grouped_fill_table(probs.data(), count, table.data());
    int64_t total = 0;
    std::memcpy(&total, table.data() + 8, sizeof(total));      // GroupedTable::total
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!staged_upload(d_table, table.data(), table.size(), st) &&
        cudaMemcpyAsync(d_table, table.data(), table.size(), cudaMemcpyHostToDevice, st) != cudaSuccess) {
        cudaGetLastError();
        return RMSMP_ERR_CUDA;
    }
    if (launch_grouped(static_cast<const uint8_t*>(d_table), table.size(), total, nt, st) != cudaSuccess) {
        cudaGetLastError();
        return RMSMP_ERR_CUDA;
    }
    return RMSMP_OK;
}

static int64_t grouped_row_blocks(const rmsmp_gemm_item* h_items, int count)
{
    int64_t n = 0;
    for (int i = 0; i < count; ++i)
        if (h_items[i].layer) n += stream_items_of(h_items[i].layer->nP, h_items[i].layer->nF4, h_items[i].layer->n8);
    return n;
}

// scratch of the E4M3 activation copies of the layers with PoT rows
static int64_t grouped_act_bytes(const rmsmp_gemm_item* h_items, int count)
{
    int64_t n = 0;
    for (int i = 0; i < count; ++i)
        if (h_items[i].layer && h_items[i].N > 0) n += stream_act_bytes(h_items[i].layer->nP, h_items[i].act_nonneg, h_items[i].N, h_items[i].layer->Kp);
    return n;
}

rmsmp_status rmsmp_grouped_plan_bytes(const rmsmp_gemm_item* h_items, int count, size_t* bytes)
{
    if (!h_items || !bytes) return RMSMP_ERR_NULL;
    if (count < 1 || count > 65536) return RMSMP_ERR_SHAPE;
    for (int i = 0; i < count; ++i) {
        if (!h_items[i].layer) return RMSMP_ERR_NULL;
        if (!layer_ok(h_items[i].layer)) return RMSMP_ERR_BAD_LAYER;
    }
    rmsmp_status a = check_arch();
    if (a != RMSMP_OK) return a;
    *bytes = stream_table_bytes(count, grouped_row_blocks(h_items, count), sm_count(), grouped_act_bytes(h_items, count));
    return RMSMP_OK;
}

rmsmp_status rmsmp_gemm_grouped_prepare(const rmsmp_gemm_item* h_items, int count, rmsmp_out_layout out_layout,
                                        void* d_table, size_t table_bytes, rmsmp_grouped_plan* plan, void* stream)
{
    NvtxRange nvtx_range("rmsmp_gemm_grouped_prepare");
    if (!d_table || !plan) return RMSMP_ERR_NULL;
    std::memset(plan, 0, sizeof(*plan));
    std::vector<Problem> probs;
    rmsmp_status s = grouped_problems(h_items, count, out_layout, probs);
    if (s != RMSMP_OK) return s;
    if ((reinterpret_cast<uintptr_t>(d_table) & 255) != 0) return RMSMP_ERR_ALIGN;
    rmsmp_status a = check_arch();
    if (a != RMSMP_OK) return a;
    for (const Problem& p : probs)
        if (!stream_supported(p)) return RMSMP_ERR_VARIANT;
    const size_t need = stream_table_bytes(count, grouped_row_blocks(h_items, count), sm_count(), grouped_act_bytes(h_items, count));
    if (table_bytes < need) return RMSMP_ERR_BUFFER_TOO_SMALL;
    const size_t head = stream_table_bytes(count, grouped_row_blocks(h_items, count), sm_count(), 0);      // the part the host fills
    std::vector<uint8_t> table(head);
    int grid = 0;
    uint32_t smem = 0, conv_grid = 0;
    if (!stream_build_table(probs.data(), count, sm_count(), table.data(), need, static_cast<uint8_t*>(d_table), &grid, &smem, &conv_grid)) return RMSMP_ERR_VARIANT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the table leaves from pageable memory: the copy has read it when the call returns
    if (cudaMemcpyAsync(d_table, table.data(), head, cudaMemcpyHostToDevice, st) != cudaSuccess) {
        cudaGetLastError();
        return RMSMP_ERR_CUDA;
    }
    plan->magic = kPlanMagicHost;
    plan->count = count;
    plan->grid = grid;
    plan->smem_bytes = smem;
    plan->conv_grid = (int32_t)conv_grid;
    plan->device = device_ordinal();
    plan->d_table = d_table;
    plan->table_bytes = need;
    return RMSMP_OK;
}

rmsmp_status rmsmp_gemm_grouped_launch(const rmsmp_grouped_plan* plan, void* stream)
{
    NvtxRange nvtx_range("rmsmp_gemm_grouped_launch");
    if (!plan) return RMSMP_ERR_NULL;
    if (plan->magic != kPlanMagicHost || !plan->d_table || plan->grid < 1) return RMSMP_ERR_BAD_LAYER;
    rmsmp_status a = check_arch();
    if (a != RMSMP_OK) return a;
    if (plan->device != device_ordinal()) return RMSMP_ERR_BAD_LAYER;
    if (plan->conv_grid < 0 || plan->conv_grid > 65535) return RMSMP_ERR_BAD_LAYER;
    if (launch_stream(static_cast<const uint8_t*>(plan->d_table), plan->grid, plan->smem_bytes, plan->count,
                      (uint32_t)plan->conv_grid, static_cast<cudaStream_t>(stream)) != cudaSuccess) {
        cudaGetLastError();
        return RMSMP_ERR_CUDA;
    }
    return RMSMP_OK;
}

rmsmp_status rmsmp_gemm_variant(const rmsmp_layer* L, const void* d_packed, const int8_t* d_act,
                                int64_t N, int64_t ld_act, float act_step, float* d_out,
                                int64_t ld_out, rmsmp_out_layout out_layout, int32_t* d_acc,
                                rmsmp_variant variant, void* stream)
{
    NvtxRange nvtx_range("rmsmp_gemm_variant");
    return gemm_impl(L, d_packed, nullptr, false, d_act, N, ld_act, act_step, d_out, ld_out, out_layout, d_acc,
                     variant, stream);
}

rmsmp_status rmsmp_gemm_workspace(const rmsmp_layer* L, const void* d_packed, const void* d_workspace,
                                  const int8_t* d_act, int64_t N, int64_t ld_act, float act_step,
                                  float* d_out, int64_t ld_out, rmsmp_out_layout out_layout,
                                  int32_t* d_acc, void* stream)
{
    NvtxRange nvtx_range("rmsmp_gemm_workspace");
    return gemm_impl(L, d_packed, d_workspace, true, d_act, N, ld_act, act_step, d_out, ld_out, out_layout,
                     d_acc, RMSMP_VARIANT_TENSOR, stream);
}

rmsmp_status rmsmp_gemm(const rmsmp_layer* L, const void* d_packed, const int8_t* d_act, int64_t N,
                        int64_t ld_act, float act_step, float* d_out, int64_t ld_out,
                        rmsmp_out_layout out_layout, int32_t* d_acc, void* stream)
{
    NvtxRange nvtx_range("rmsmp_gemm");
    return rmsmp_gemm_variant(L, d_packed, d_act, N, ld_act, act_step, d_out, ld_out, out_layout,
                              d_acc, RMSMP_VARIANT_AUTO, stream);
}

static rmsmp_status conv_impl(const rmsmp_layer* L, const void* d_packed, const void* d_ws, bool use_ws,
                              const int8_t* d_act, int B, int H, int W, int stride, int pad, float act_step,
                              float* d_out, rmsmp_out_layout out_layout, int32_t* d_acc,
                              rmsmp_variant variant, void* stream, const Requant* rq = nullptr)
{
    if (!L || !d_packed || !d_act || (!d_out && !rq) || (use_ws && !d_ws)) return RMSMP_ERR_NULL;
    if (!layer_ok(L)) return RMSMP_ERR_BAD_LAYER;
    if (B < 1 || H < 1 || W < 1 || stride < 1 || stride > 8 || pad < 0 || pad > 16) return RMSMP_ERR_SHAPE;
    if (H + 2 * pad < L->kh || W + 2 * pad < L->kw) return RMSMP_ERR_SHAPE;
    if (out_layout != RMSMP_OUT_NM && out_layout != RMSMP_OUT_MN) return RMSMP_ERR_SHAPE;
    if (!std::isfinite(act_step)) return RMSMP_ERR_SCALE;
    const int Ho = (H + 2 * pad - L->kh) / stride + 1, Wo = (W + 2 * pad - L->kw) / stride + 1;
    const int64_t N = (int64_t)B * Ho * Wo;
    if (N > (int64_t)1 << 31 || (int64_t)B * H * W > (int64_t)1 << 31) return RMSMP_ERR_SHAPE;
    if (!aligned16(d_act) || (!rq && !aligned16(d_out)) || (d_acc && !aligned16(d_acc)) ||
        (reinterpret_cast<uintptr_t>(d_packed) & 255))
        return RMSMP_ERR_ALIGN;
    rmsmp_status a = check_arch();
    if (a != RMSMP_OK) return a;
    Problem p;
    fill_problem(p, L, d_packed);
    p.act = d_act;
    p.B = B; p.H = H; p.W = W; p.Ho = Ho; p.Wo = Wo; p.stride = stride; p.pad = pad;
    p.pix_pitch = L->Cin; p.N = N;
    p.act_step = act_step; p.out = d_out; p.acc = d_acc;
    p.out_mn = (out_layout == RMSMP_OUT_MN);
    p.ld_out = p.out_mn ? N : L->M;
    if (rq) { p.rq_codes = rq->codes; p.rq_alpha = rq->alpha; p.rq_kind = rq->kind; p.ld_codes = L->M; }
    if (use_ws) {
        if (!aligned16(d_ws)) return RMSMP_ERR_ALIGN;
        p.wexp = static_cast<const int8_t*>(d_ws);
    }
    return dispatch(p, variant, static_cast<cudaStream_t>(stream));
}

rmsmp_status rmsmp_conv_depthwise(const rmsmp_layer* L, const void* d_packed, const int8_t* d_act, int B, int H, int W,
                                  int stride, int pad, float act_step, float* d_out, int32_t* d_acc, void* stream)
{
    NvtxRange nvtx_range("rmsmp_conv_depthwise");
    if (!L || !d_packed || !d_act || !d_out) return RMSMP_ERR_NULL;
    if (!layer_ok(L)) return RMSMP_ERR_BAD_LAYER;
    if (L->Cin != 1) return RMSMP_ERR_SHAPE;              // a depthwise layer is described as M = channels, Cin = 1
    if (B < 1 || H < 1 || W < 1 || stride < 1 || stride > 8 || pad < 0 || pad > 16) return RMSMP_ERR_SHAPE;
    if (H + 2 * pad < L->kh || W + 2 * pad < L->kw) return RMSMP_ERR_SHAPE;
    if (!std::isfinite(act_step)) return RMSMP_ERR_SCALE;
    const int Ho = (H + 2 * pad - L->kh) / stride + 1, Wo = (W + 2 * pad - L->kw) / stride + 1;
    const int64_t N = (int64_t)B * Ho * Wo;
    if (N > (int64_t)1 << 31 || (int64_t)B * H * W > (int64_t)1 << 31) return RMSMP_ERR_SHAPE;
    if (!aligned16(d_act) || !aligned16(d_out) || (d_acc && !aligned16(d_acc)) || (reinterpret_cast<uintptr_t>(d_packed) & 255))
        return RMSMP_ERR_ALIGN;
    rmsmp_status a = check_arch();
    if (a != RMSMP_OK) return a;
    Problem p;
    fill_problem(p, L, d_packed);
    p.act = d_act;
    p.B = B; p.H = H; p.W = W; p.Ho = Ho; p.Wo = Wo; p.stride = stride; p.pad = pad;
    p.pix_pitch = L->M; p.N = N;                          // channels last: a pixel holds one code per channel
    p.act_step = act_step; p.out = d_out; p.acc = d_acc; p.out_mn = 0; p.ld_out = L->M;
    if (!depthwise_supported(p)) return RMSMP_ERR_VARIANT;
    if (launch_depthwise(p, static_cast<cudaStream_t>(stream)) != cudaSuccess) {
        cudaGetLastError();
        return RMSMP_ERR_CUDA;
    }
    return RMSMP_OK;
}

rmsmp_status rmsmp_im2col_codes(const int8_t* d_act, int B, int H, int W, int C, int64_t pix_pitch, int kh, int kw,
                                int stride, int pad, int8_t* d_cols, int64_t ld_cols, void* stream)
{
    NvtxRange nvtx_range("rmsmp_im2col_codes");
    if (!d_act || !d_cols) return RMSMP_ERR_NULL;
    if (B < 1 || H < 1 || W < 1 || C < 1 || C > 64 || kh < 1 || kw < 1 || kh > 16 || kw > 16) return RMSMP_ERR_SHAPE;
    if (stride < 1 || stride > 8 || pad < 0 || pad > 16 || pix_pitch < C) return RMSMP_ERR_SHAPE;
    if (H + 2 * pad < kh || W + 2 * pad < kw) return RMSMP_ERR_SHAPE;
    if (ld_cols < (int64_t)kh * kw * C || ld_cols > 4096) return RMSMP_ERR_SHAPE;
    const int Ho = (H + 2 * pad - kh) / stride + 1, Wo = (W + 2 * pad - kw) / stride + 1;
    if ((int64_t)B * Ho * Wo > (int64_t)1 << 31 || (int64_t)B * H * W > (int64_t)1 << 31) return RMSMP_ERR_SHAPE;
    if (!aligned16(d_cols) || (ld_cols & 15)) return RMSMP_ERR_ALIGN;
    rmsmp_status a = check_arch();
    if (a != RMSMP_OK) return a;
    if (launch_im2col(d_act, B, H, W, C, pix_pitch, kh, kw, stride, pad, Ho, Wo, d_cols, ld_cols,
                      static_cast<cudaStream_t>(stream)) != cudaSuccess) {
        cudaGetLastError();
        return RMSMP_ERR_CUDA;
    }
    return RMSMP_OK;
}

rmsmp_status rmsmp_conv_implicit_variant(const rmsmp_layer* L, const void* d_packed,
                                         const int8_t* d_act, int B, int H, int W, int stride,
                                         int pad, float act_step, float* d_out,
                                         rmsmp_out_layout out_layout, int32_t* d_acc,
                                         rmsmp_variant variant, void* stream)
{
    NvtxRange nvtx_range("rmsmp_conv_implicit_variant");
    return conv_impl(L, d_packed, nullptr, false, d_act, B, H, W, stride, pad, act_step, d_out, out_layout,
                     d_acc, variant, stream);
}

rmsmp_status rmsmp_conv_implicit_workspace(const rmsmp_layer* L, const void* d_packed,
                                           const void* d_workspace, const int8_t* d_act, int B, int H,
                                           int W, int stride, int pad, float act_step, float* d_out,
                                           rmsmp_out_layout out_layout, int32_t* d_acc, void* stream)
{
    NvtxRange nvtx_range("rmsmp_conv_implicit_workspace");
    return conv_impl(L, d_packed, d_workspace, true, d_act, B, H, W, stride, pad, act_step, d_out, out_layout,
                     d_acc, RMSMP_VARIANT_TENSOR, stream);
}

rmsmp_status rmsmp_gemm_workspace_requant(const rmsmp_layer* L, const void* d_packed, const void* d_workspace,
                                          const int8_t* d_act, int64_t N, int64_t ld_act, float act_step,
                                          float next_alpha, rmsmp_act_kind next_kind, int8_t* d_next_codes,
                                          int64_t ld_codes, float* h_next_step, void* stream)
{
    NvtxRange nvtx_range("rmsmp_gemm_workspace_requant");
    const Requant rq = {next_alpha, next_kind, d_next_codes, ld_codes};
    rmsmp_status s = requant_check(&rq, h_next_step);
    if (s != RMSMP_OK) return s;
    return gemm_impl(L, d_packed, d_workspace, true, d_act, N, ld_act, act_step, nullptr, 0, RMSMP_OUT_NM, nullptr,
                     RMSMP_VARIANT_TENSOR, stream, &rq);
}

rmsmp_status rmsmp_conv_implicit_workspace_requant(const rmsmp_layer* L, const void* d_packed,
                                                   const void* d_workspace, const int8_t* d_act, int B, int H,
                                                   int W, int stride, int pad, float act_step, float next_alpha,
                                                   rmsmp_act_kind next_kind, int8_t* d_next_codes,
                                                   float* h_next_step, void* stream)
{
    NvtxRange nvtx_range("rmsmp_conv_implicit_workspace_requant");
    const Requant rq = {next_alpha, next_kind, d_next_codes, 0};
    rmsmp_status s = requant_check(&rq, h_next_step);
    if (s != RMSMP_OK) return s;
    return conv_impl(L, d_packed, d_workspace, true, d_act, B, H, W, stride, pad, act_step, nullptr, RMSMP_OUT_NM,
                     nullptr, RMSMP_VARIANT_TENSOR, stream, &rq);
}

rmsmp_status rmsmp_workspace_bytes(const rmsmp_layer* L, size_t* bytes)
{
    if (!L || !bytes) return RMSMP_ERR_NULL;
    if (!layer_ok(L)) return RMSMP_ERR_BAD_LAYER;
    *bytes = (size_t)align_up((uint64_t)L->M * L->Kp, 256);
    return RMSMP_OK;
}

rmsmp_status rmsmp_expand_weights(const rmsmp_layer* L, const void* d_packed, void* d_workspace,
                                  size_t workspace_bytes, void* stream)
{
    NvtxRange nvtx_range("rmsmp_expand_weights");
    if (!L || !d_packed || !d_workspace) return RMSMP_ERR_NULL;
    if (!layer_ok(L)) return RMSMP_ERR_BAD_LAYER;
    if (workspace_bytes < (size_t)L->M * L->Kp) return RMSMP_ERR_BUFFER_TOO_SMALL;
    if (!aligned16(d_workspace) || (reinterpret_cast<uintptr_t>(d_packed) & 255)) return RMSMP_ERR_ALIGN;
    rmsmp_status a = check_arch();
    if (a != RMSMP_OK) return a;
    if (launch_expand(*L, static_cast<const uint8_t*>(d_packed), static_cast<int8_t*>(d_workspace),
                      static_cast<cudaStream_t>(stream)) != cudaSuccess) {
        cudaGetLastError();
        return RMSMP_ERR_CUDA;
    }
    return RMSMP_OK;
}

rmsmp_status rmsmp_conv_implicit(const rmsmp_layer* L, const void* d_packed, const int8_t* d_act,
                                 int B, int H, int W, int stride, int pad, float act_step,
                                 float* d_out, rmsmp_out_layout out_layout, int32_t* d_acc,
                                 void* stream)
{
    NvtxRange nvtx_range("rmsmp_conv_implicit");
    return rmsmp_conv_implicit_variant(L, d_packed, d_act, B, H, W, stride, pad, act_step, d_out,
                                       out_layout, d_acc, RMSMP_VARIANT_AUTO, stream);
}

rmsmp_status rmsmp_last_device_status(const void* d_packed, void* stream)
{
    if (!d_packed) return RMSMP_ERR_NULL;
    uint32_t w = 0;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(&w, static_cast<const uint8_t*>(d_packed) + kStatusOffset, 4,
                        cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) {
        cudaGetLastError();
        return RMSMP_ERR_CUDA;
    }
    return w <= RMSMP_ERR_VARIANT ? (rmsmp_status)w : RMSMP_ERR_CUDA;
}

}  // extern "C"
