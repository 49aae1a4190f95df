/*
 * rmsmp.h -- C ABI of the B200 (sm_100a) RMSMP layer library.
 *
 * The library runs the inference arithmetic of one linear or convolution layer quantized
 * the RMSMP way (paper Section 3): every weight row (= output feature / filter) carries
 * its own scheme and precision -- Power-of-Two 4-bit, Fixed-point 4-bit or Fixed-point
 * 8-bit, in a per-layer ratio fixed offline -- and multiplies 4-bit fixed-point
 * activations.  Integer accumulation is exact; the output is rescaled per row.
 *
 * Conventions
 *   - Pointers named d_* are DEVICE pointers, h_* are HOST pointers.  The caller owns every
 *     buffer; the library allocates no device memory and keeps no reference after a call
 *     returns (work already queued on the stream keeps using the buffers until it is done).
 *     The only memory it obtains by itself is 2 MiB of pinned HOST memory per device, on the first
 *     rmsmp_quantize_pack, used to upload the layer metadata without stalling the stream.
 *   - `stream` is a cudaStream_t passed as void* (0 = default stream).  All device work is
 *     asynchronous on it.
 *   - Every function returns an rmsmp_status and never throws, aborts or prints.  Everything
 *     that can be validated on the host is validated before anything is launched.
 *   - Device pointers must be 16-byte aligned unless stated otherwise.
 */
#ifndef RMSMP_H_
#define RMSMP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    RMSMP_OK = 0,
    RMSMP_ERR_NULL = 1,             /* a required pointer is NULL */
    RMSMP_ERR_SHAPE = 2,            /* a dimension is < 1 or beyond the supported range */
    RMSMP_ERR_SCHEME = 3,           /* (scheme, bits) not one of PoT-4, Fixed-4, Fixed-8 */
    RMSMP_ERR_SCALE = 4,            /* a clip value alpha is not finite and > 0 */
    RMSMP_ERR_ALIGN = 5,            /* pointer or leading dimension not 16-byte aligned */
    RMSMP_ERR_BUFFER_TOO_SMALL = 6, /* packed buffer smaller than rmsmp_layer.packed_bytes */
    RMSMP_ERR_ARCH = 7,             /* current device is not compute capability 10.x */
    RMSMP_ERR_CUDA = 8,             /* a CUDA runtime/driver call failed */
    RMSMP_ERR_TIMEOUT = 9,          /* a bounded in-kernel wait ran out (device status word) */
    RMSMP_ERR_BAD_LAYER = 10,       /* rmsmp_layer not produced by rmsmp_layer_init */
    RMSMP_ERR_VARIANT = 11          /* requested kernel variant cannot run this problem */
} rmsmp_status;

/* The scheme/precision menu of the method (Figure 2): bits is 4 or 8; PoT only with 4. */
typedef enum { RMSMP_SCHEME_POT = 0, RMSMP_SCHEME_FIXED = 1 } rmsmp_scheme;
/* Activation codes: unsigned 4-bit (0..15, post-ReLU inputs) or symmetric signed (-7..7). */
typedef enum { RMSMP_ACT_U4 = 0, RMSMP_ACT_S4 = 1 } rmsmp_act_kind;
/* PoT rounding: nearest level of Eq. 4 (default) or the printed 2^round(log2 x) rule of Eq. 5. */
typedef enum { RMSMP_POT_NEAREST = 0, RMSMP_POT_LOG2 = 1 } rmsmp_pot_mode;
/* Output layout: y[n*ld + m] (pixels/tokens major, default) or y[m*ld + n]. */
typedef enum { RMSMP_OUT_NM = 0, RMSMP_OUT_MN = 1 } rmsmp_out_layout;
/* Weight source layout: [M][K] row-major, or filters [M][Cin][kh][kw]. */
typedef enum { RMSMP_W_LINEAR = 0, RMSMP_W_CONV_OIHW = 1 } rmsmp_w_layout;
/* Which kernel carries out the contraction. */
typedef enum {
    RMSMP_VARIANT_AUTO = 0,      /* library picks by shape */
    RMSMP_VARIANT_TENSOR = 1,    /* TMA + in-smem code expansion + tcgen05 int8 MMA, TMEM accumulators.  A layer of one
                                    128-row block whose expanded weights fit 72 KB is expanded ONCE per CTA into
                                    resident shared memory; longer rows are expanded k-block by k-block per tile */
    RMSMP_VARIANT_SIMT = 2,      /* CUDA-core integer multiply-add (dp4a) on codes expanded in registers */
    RMSMP_VARIANT_SHIFTADD = 3,  /* CUDA cores; PoT rows by shift-and-add, no multiplier */
    RMSMP_VARIANT_SIMPLE = 4     /* one thread per output, scalar; bring-up / cross-check */
} rmsmp_variant;

/*
 * Host-side description of one packed layer.  Filled by rmsmp_layer_init from the shape and
 * the per-row scheme map; plain data, may be copied or stored with the packed buffer.
 * The packed buffer itself is position independent.
 *
 * Packed buffer layout (offsets in bytes from its start, every section 256-byte aligned):
 *   header (256 B: magic, version, dims, counts; device status word at byte 64)
 *   perm  [M] int32   packed position -> original row; PoT-4 rows, then Fixed-4, then
 *                     Fixed-8, each group in original order (stable)
 *   slot  [M] int32   original row -> packed position
 *   wstep [M] float   by original row: real weight = integer value * wstep
 *   alpha [M] float   by original row: clip value used by the quantizer
 *   kind  [M] uint8   by original row: 0 PoT-4, 1 Fixed-4, 2 Fixed-8
 *   blocks[ceil(M/128)][8] int32: for each block of 128 original rows the first packed
 *                     position and count of its PoT-4, Fixed-4 and Fixed-8 rows
 *                     {p0, nP, f0, nF, e0, nE, 0, 0} (positions relative to each group)
 *   q4    [(nP+nF4)][Kp/2] bytes: 4-bit codes, two per byte
 *   q8    [n8][Kp] bytes: int8 codes
 * Reduction index inside a packed row: k' = (i*kw + j)*Cp + c  (tap-major, channels last),
 * Cp = Cin rounded up to 32, Kp = kh*kw*Cp rounded up to 128; pad codes are zero.
 * Inside each aligned group of 32 codes (16 bytes): PoT-4 stores code 2b in the low and
 * 2b+1 in the high nibble of byte b (nibble = sign<<3 | e, value 0 or +-2^(e-1));
 * Fixed-4 stores code b in the high and code 16+b in the low nibble of byte b
 * (two's complement).
 */
typedef struct rmsmp_layer {
    uint32_t magic;             /* set by rmsmp_layer_init */
    int32_t M, Cin, kh, kw;     /* rows; reduction length K = Cin*kh*kw (linear: kh = kw = 1) */
    int32_t Cp, Kp;             /* padded channel count per tap, padded packed row length */
    int32_t nP, nF4, n8;        /* rows per group */
    int32_t nblocks;            /* ceil(M/128) */
    int32_t raw_stage_bytes;    /* shared-memory bytes the packed codes of one 128-row block's k-block need (tensor kernel) */
    uint64_t off_perm, off_slot, off_wstep, off_alpha, off_kind, off_blocks, off_q4, off_q8;
    uint64_t packed_bytes;      /* size the packed buffer must have */
} rmsmp_layer;

const char* rmsmp_status_string(rmsmp_status s);

/*
 * Host helper: scheme/precision map of a layer from the ratio PoT-4 : Fixed-4 : Fixed-8 =
 * A : B : C (Section 3.3, A + B + C = 100; Section 3.1: lower variance -> PoT).
 * n8 = floor(M*C/100 + 1/2) rows of HIGHEST variance get Fixed-8 (a stand-in for the
 * Hessian ranking of Algorithm 1, which needs a loss), of the rest the nP = floor(M*A/100
 * + 1/2) rows of LOWEST variance get PoT-4, the others Fixed-4.  Ranking key: (population
 * variance in double, row index).  h_W is [M][K] fp32 on the host; h_scheme / h_bits
 * receive M entries.  Errors: NULL, SHAPE (M, K < 1 or A + B + C != 100 or negative).
 */
rmsmp_status rmsmp_assign_rows(const float* h_W, int M, int K, int A, int B, int C,
                               uint8_t* h_scheme, uint8_t* h_bits);

/*
 * Describe a layer: counts rows per group, lays out the packed buffer, sets
 * layer->packed_bytes.  Host only; no CUDA call.  Limits: 1 <= M <= 2^20,
 * 1 <= Cin*kh*kw <= 1,000,000 (keeps |sum| < 2^31), kh, kw <= 16.
 * Errors: NULL, SHAPE, SCHEME (an entry outside {PoT-4, Fixed-4, Fixed-8}; PoT-8 is not in
 * the method, Section 3.2).
 */
rmsmp_status rmsmp_layer_init(rmsmp_layer* layer, int M, int Cin, int kh, int kw,
                              const uint8_t* h_scheme, const uint8_t* h_bits);

/*
 * Quantize and pack the weights (Eq. 1-5; grouping by scheme, Section 3.1 / 4.1).
 * d_W: fp32 weights on the device, [M][K] (RMSMP_W_LINEAR) or [M][Cin][kh][kw]
 * (RMSMP_W_CONV_OIHW), 16-byte aligned.  h_scheme/h_bits/h_alpha: M host entries each
 * (the assignment and the clip values are offline decisions).  Quantizers, per row r with
 * t = clip(w / alpha_r, -1, 1) in fp32:
 *   Fixed-m: q = round_half_even(t * (2^(m-1)-1)), weight = q * alpha_r/(2^(m-1)-1)
 *   PoT-4:   sign/exponent code of the nearest level of +-{0, 2^-6..2^0} (ties to the larger
 *            magnitude), or of 2^round(log2|t|) in RMSMP_POT_LOG2 mode; weight = v * alpha_r/64
 * Writes layer->packed_bytes bytes to d_packed (256-byte aligned) and clears its status word.
 * Errors: NULL, BAD_LAYER, SCHEME (map differs from the one given to rmsmp_layer_init),
 * SCALE, ALIGN, BUFFER_TOO_SMALL, ARCH, CUDA.
 */
rmsmp_status rmsmp_quantize_pack(const float* d_W, rmsmp_w_layout w_layout,
                                 const rmsmp_layer* layer, const uint8_t* h_scheme,
                                 const uint8_t* h_bits, const float* h_alpha,
                                 rmsmp_pot_mode pot_mode, void* d_packed, size_t packed_bytes,
                                 void* stream);

/*
 * The same from the ratio alone: the row assignment runs on the device (Section 3.1: of two rows
 * the one with the lower variance takes PoT; Section 3.3: ratio PoT-4 : Fixed-4 : Fixed-8 = A : B : C;
 * Algorithm 1's assignment block, with the variance rank standing in for its Hessian ranking as in
 * rmsmp_assign_rows), so nothing about the weights has to be known on the host.
 *   rmsmp_layer_init_ratio       describes the layer from the ratio: the row counts per kind follow
 *                                from M and A:B:C (n8 = floor(M*C/100 + 1/2), nP = floor(M*A/100 + 1/2),
 *                                the rest Fixed-4), which fixes the packed layout.  Host only.  M <= 65536.
 *   rmsmp_assign_scratch_bytes   device scratch the assignment needs (16 bytes per row).
 *   rmsmp_assign_quantize_pack   per-row population variance (double, two passes in reduction order),
 *                                rank by (variance, row index), kinds from the rank, stable grouping,
 *                                all metadata of the packed buffer, then the quantizers of
 *                                rmsmp_quantize_pack.  d_alpha: M clip values on the device, or NULL for
 *                                alpha_r = max |w| of the row (1 for an all-zero row).  d_scheme / d_bits
 *                                (optional, M bytes each on the device) receive the assignment.  The
 *                                result equals rmsmp_assign_rows + rmsmp_quantize_pack bit for bit.
 * Errors: NULL, BAD_LAYER, SHAPE, SCHEME (descriptor built for another ratio), BUFFER_TOO_SMALL, ALIGN,
 * ARCH, CUDA.
 */
rmsmp_status rmsmp_layer_init_ratio(rmsmp_layer* layer, int M, int Cin, int kh, int kw, int A, int B, int C);
rmsmp_status rmsmp_assign_scratch_bytes(int M, size_t* bytes);
rmsmp_status rmsmp_assign_quantize_pack(const float* d_W, rmsmp_w_layout w_layout, const rmsmp_layer* layer,
                                        int A, int B, int C, const float* d_alpha, rmsmp_pot_mode pot_mode,
                                        void* d_packed, size_t packed_bytes, void* d_scratch, size_t scratch_bytes,
                                        uint8_t* d_scheme, uint8_t* d_bits, void* stream);

/*
 * Parity/debug (checks the level sets of Eq. 1 and Eq. 4 and the row grouping of Section 3.1 /
 * 4.1 from outside): expand a packed buffer back to integer values in ORIGINAL row order and
 * original reduction order ([M][K], conv: [M][Cin][kh][kw]); Fixed rows give q, PoT rows
 * 0 or +-2^(e-1).  d_perm (packed -> original, M int32) and d_wstep (by original row,
 * M floats) may be NULL.  Errors: NULL, BAD_LAYER, ARCH, CUDA.
 */
rmsmp_status rmsmp_unpack_codes(const rmsmp_layer* layer, const void* d_packed,
                                int8_t* d_values, int32_t* d_perm, float* d_wstep,
                                void* stream);

/*
 * 4-bit activation quantizer (Section 3.1: activations are Fixed 4-bit for every row kind).
 * One clip value per tensor.  U4: a = round_half_even(clip(x/alpha_a, 0, 1) * 15), step
 * alpha_a/15.  S4: Fixed-4 of Eq. 1 with alpha_a, step alpha_a/7.  d_X: `count` floats;
 * d_codes: `count` int8 (one code per byte).  *h_act_step receives the step (host, may be
 * NULL).  Infinite inputs clip like any other value; the code of a NaN input is unspecified.
 * Pointers need only their natural alignment.  Errors: NULL, SHAPE, SCALE, ARCH, CUDA.
 */
rmsmp_status rmsmp_quantize_act(const float* d_X, size_t count, float alpha_a,
                                rmsmp_act_kind kind, int8_t* d_codes, float* h_act_step,
                                void* stream);

/*
 * Linear layer (Algorithm 1, forward line): for every token n and row m
 *   acc[n][m] = sum_k value[m][k] * act[n][k]          (int32, exact)
 *   y[n][m]   = (float)acc[n][m] * (wstep[m] * act_step)
 * d_act: int8 codes [N][ld_act], ld_act >= K and a multiple of 16.  d_out: fp32, layout
 * `out_layout` with leading dimension ld_out (>= M for NM, >= N for MN).  d_acc (optional,
 * may be NULL): int32 accumulators in the same layout and leading dimension.
 * layer must describe a linear layer (kh = kw = 1).
 * Errors: NULL, BAD_LAYER, SHAPE, ALIGN, ARCH, VARIANT, CUDA.
 */
rmsmp_status rmsmp_gemm(const rmsmp_layer* layer, const void* d_packed, const int8_t* d_act,
                        int64_t N, int64_t ld_act, float act_step, float* d_out,
                        int64_t ld_out, rmsmp_out_layout out_layout, int32_t* d_acc,
                        void* stream);
rmsmp_status rmsmp_gemm_variant(const rmsmp_layer* layer, const void* d_packed,
                                const int8_t* d_act, int64_t N, int64_t ld_act, float act_step,
                                float* d_out, int64_t ld_out, rmsmp_out_layout out_layout,
                                int32_t* d_acc, rmsmp_variant variant, void* stream);

/*
 * Convolution layer (Algorithm 1's forward line with filters as the weight rows: Section 3,
 * Figure 2 -- every filter carries its own scheme and precision) as an implicit GEMM (no im2col
 * buffer): activation codes d_act are
 * [B][H][W][Cin] (channels last), zero outside the image; output pixel index
 * n = (b*Ho + ho)*Wo + wo with Ho = (H + 2*pad - kh)/stride + 1 (same for Wo); results as in
 * rmsmp_gemm with N = B*Ho*Wo and dense leading dimension (M for NM, N for MN).
 * Errors: NULL, BAD_LAYER, SHAPE, ALIGN (Cin not a multiple of 16 for the tensor variant
 * selects another variant under AUTO, and is VARIANT when RMSMP_VARIANT_TENSOR is forced),
 * ARCH, VARIANT, CUDA.
 */
rmsmp_status rmsmp_conv_implicit(const rmsmp_layer* layer, const void* d_packed,
                                 const int8_t* d_act, int B, int H, int W, int stride, int pad,
                                 float act_step, float* d_out, rmsmp_out_layout out_layout,
                                 int32_t* d_acc, void* stream);
rmsmp_status rmsmp_conv_implicit_variant(const rmsmp_layer* layer, const void* d_packed,
                                         const int8_t* d_act, int B, int H, int W, int stride,
                                         int pad, float act_step, float* d_out,
                                         rmsmp_out_layout out_layout, int32_t* d_acc,
                                         rmsmp_variant variant, void* stream);

/*
 * Depthwise convolution (the 3x3 layers of MobileNet-v2, one of the paper's models, Section 4.1): every
 * channel is convolved with its own filter, and every filter is a weight row with its own scheme and
 * precision (Figure 2).  The layer is described and packed like any other with M = channels and Cin = 1
 * (weights [C][1][kh][kw]); activation codes d_act are [B][H][W][C], results
 *   acc[b][ho][wo][c] = sum_{i,j} value[c][i][j] * act[b][ho*stride+i-pad][wo*stride+j-pad][c]   (zero outside)
 *   y = (float)acc * (wstep[c] * act_step)
 * in [B][Ho][Wo][C]; d_acc optional.  CUDA cores (there is no contraction over channels).
 * Errors: NULL, BAD_LAYER, SHAPE (layer not Cin = 1, bad geometry), SCALE, ALIGN, ARCH, CUDA; VARIANT when C is
 * not a multiple of 4 or the filters do not fit shared memory (kh * kw * C > 51,200).
 */
rmsmp_status rmsmp_conv_depthwise(const rmsmp_layer* layer, const void* d_packed, const int8_t* d_act, int B,
                                  int H, int W, int stride, int pad, float act_step, float* d_out,
                                  int32_t* d_acc, void* stream);

/*
 * Patch matrix of a convolution with few input channels (a network's first layer: 3 channels,
 * 7 x 7 filters, stride 2; Section 4.1 and Table 6 quantize that layer like all others).  The
 * implicit form fetches one filter tap per bulk copy, which needs 16 bytes of channels per pixel;
 * a 3-channel layer is instead run as a linear layer over its patches:
 *   d_cols[n][(i * kw + j) * C + c] = d_act[b][ho * stride + i - pad][wo * stride + j - pad][c]
 * for output pixel n = (b * Ho + ho) * Wo + wo, zero outside the image and in the columns from
 * kh * kw * C up to ld_cols.  The layer's weights are packed as a linear layer with K = ld_cols
 * in the same order ([M][kh][kw][C], zero columns appended), and rmsmp_gemm* on d_cols with
 * N = B * Ho * Wo gives the convolution's [N][M] output.
 *   d_act    device, int8 codes [B][H][W] pixels of pix_pitch bytes, the first C of which are used
 *   d_cols   device, 16-byte aligned, [B*Ho*Wo][ld_cols]; ld_cols a multiple of 16, >= kh*kw*C
 * Limits: C <= 64, kh, kw <= 16, stride 1..8, pad 0..16, ld_cols <= 4096.  Allocates nothing; one kernel
 * on `stream`.
 * Errors: NULL, SHAPE (limits, ld_cols too small, more than 2^31 pixels), ALIGN, ARCH, CUDA.
 */
rmsmp_status rmsmp_im2col_codes(const int8_t* d_act, int B, int H, int W, int C, int64_t pix_pitch,
                                int kh, int kw, int stride, int pad, int8_t* d_cols, int64_t ld_cols,
                                void* stream);

/*
 * Many small-batch linear layers in one launch (Algorithm 1's forward line, layer after layer;
 * Section 3.1: the layers execute one after another on the same hardware).  With a
 * handful of tokens a layer is bound by reading its packed weights once, which takes a fraction
 * of a microsecond -- less than a kernel launch -- so the layers are handed over together and one
 * kernel streams all their weights.  Every item is computed exactly as rmsmp_gemm would (CUDA
 * cores, codes expanded in registers).  Items must not write to memory another item reads
 * (they run concurrently).
 *   h_items   `count` host structures (1 <= count <= 65536), all linear layers.
 *   d_table   device scratch of rmsmp_grouped_table_bytes(count) bytes, 16-byte aligned; the
 *             library writes the problem table there (it must stay untouched until the work
 *             queued by this call has finished).
 * Errors: as rmsmp_gemm per item, BUFFER_TOO_SMALL for the table.
 */
typedef struct rmsmp_gemm_item {
    const rmsmp_layer* layer;
    const void* d_packed;
    const int8_t* d_act;       /* [N][ld_act] */
    int64_t N, ld_act;
    float act_step;
    float* d_out;
    int64_t ld_out;
    int32_t* d_acc;            /* optional */
    int32_t act_nonneg;        /* tensor-core grouped launch only: nonzero = the caller guarantees that every
                                  activation code is within 0..15 (the unsigned 4-bit activations of Eq. 1);
                                  0 = codes may be negative (within -16..16) */
} rmsmp_gemm_item;
rmsmp_status rmsmp_grouped_table_bytes(int count, size_t* bytes);
rmsmp_status rmsmp_gemm_grouped(const rmsmp_gemm_item* h_items, int count, rmsmp_out_layout out_layout,
                                void* d_table, size_t table_bytes, void* stream);

/*
 * The same grouped launch on the tensor cores, split into a set-up call and a launch call
 * (Section 3.1: rows of every scheme streamed to their cores and finishing together; here all
 * layers' packed rows stream through the SMs in one kernel).  One persistent CTA per SM takes
 * blocks of 128 rows of one kind of any layer, fetches their packed codes with TMA, expands them
 * in registers, hands them to the tensor cores through tensor memory and multiplies them with up
 * to 128 tokens on tcgen05.  Fixed-4 and Fixed-8 rows become int8 operands with int32 sums.  A
 * PoT-4 code (Eq. 4: sign and exponent) shifted left by two is the 6-bit float of a quarter of its
 * value, so PoT rows go to the tensor core's float path as they are (E3M2 weights x E4M3
 * activations, fp32 sums); every product and partial sum is a multiple of 1/4 below 2^22, which
 * fp32 holds exactly.  The activation bytes of a layer whose item says act_nonneg are read as
 * they are: a byte 0..15 taken as an E4M3 number is that code times 2^-9.  Otherwise the launch
 * first writes an E4M3 copy of the layer's codes into scratch behind the table.  Results are bit
 * for bit those of rmsmp_gemm for activation codes within -16..16 (the 4-bit codes of Eq. 1/Eq. 3,
 * signed or unsigned; 0..15 with act_nonneg); other int8 values are not supported by this entry
 * point.
 *   rmsmp_grouped_plan_bytes    scratch size for the table of these layers on the current device
 *                               (the table proper plus N x K bytes per layer with PoT rows and
 *                               without act_nonneg for the E4M3 copy of its activation codes, which
 *                               every launch rewrites).
 *   rmsmp_gemm_grouped_prepare  validates the items, builds the table (tensor maps of every
 *                               layer's packed rows and activations, work lists per SM) and queues
 *                               its upload to d_table (256-byte aligned) on `stream`; fills *plan.
 *                               Every item needs N <= 128, and K <= 16384 if it has PoT rows (the
 *                               exactness bound of the fp32 sums), else RMSMP_ERR_VARIANT.  The call costs
 *                               host time proportional to the number of layers: do it once.
 *   rmsmp_gemm_grouped_launch   one launch from a prepared plan (the streaming kernel, behind a small
 *                               kernel that writes the activation copies); may be repeated for as
 *                               long as the buffers, shapes and leading dimensions the plan was
 *                               built from stay the same (their CONTENTS may change: new weights
 *                               packed with the same row map, new activation codes).  The table
 *                               must stay untouched while launches that use it are in flight.  The
 *                               kernels are launched with the programmatic-stream-serialization
 *                               attribute and signal early, so that launches in a row overlap their
 *                               ends and beginnings; what a predecessor may still touch is accessed only
 *                               behind a grid-dependency wait.  Kernels that follow on the stream and
 *                               are launched the ordinary way are ordered as always; one that is itself
 *                               launched with that attribute must call cudaGridDependencySynchronize()
 *                               before it reads the results.
 * Errors: as rmsmp_gemm_grouped; BAD_LAYER for a plan that was not prepared, or was prepared on
 * another device.
 */
typedef struct rmsmp_grouped_plan {
    uint32_t magic;            /* set by rmsmp_gemm_grouped_prepare */
    int32_t count;             /* layers */
    int32_t grid;              /* CTAs of the launch */
    uint32_t smem_bytes;       /* dynamic shared memory per CTA */
    int32_t device;            /* ordinal of the device the table was built for */
    int32_t conv_grid;         /* blocks per layer of the kernel that writes the E4M3 activation copies (0: no PoT rows) */
    const void* d_table;
    uint64_t table_bytes;
} rmsmp_grouped_plan;
rmsmp_status rmsmp_grouped_plan_bytes(const rmsmp_gemm_item* h_items, int count, size_t* bytes);
rmsmp_status rmsmp_gemm_grouped_prepare(const rmsmp_gemm_item* h_items, int count, rmsmp_out_layout out_layout,
                                        void* d_table, size_t table_bytes, rmsmp_grouped_plan* plan,
                                        void* stream);
rmsmp_status rmsmp_gemm_grouped_launch(const rmsmp_grouped_plan* plan, void* stream);

/*
 * Workspace variant of the tensor-core path.  The expansion of the 4-bit / PoT codes to int8
 * (the GPU counterpart of routing rows to the per-scheme GEMM cores, Section 4.1) is done ONCE
 * per layer into caller-provided scratch memory instead of once per output tile in shared
 * memory; the contraction kernel then fetches plain int8 rows with TMA.  Same results bit for
 * bit.  Worth it when N is large (the expansion is amortised over all pixels).
 *   rmsmp_workspace_bytes   size of the scratch buffer for a layer (M * Kp bytes, rounded up).
 *   rmsmp_expand_weights    fills d_workspace ([M][Kp] int8 values, original row order, packed
 *                           reduction order) from the packed buffer; must be repeated whenever
 *                           the packed buffer changes.  d_workspace: 16-byte aligned.
 *   rmsmp_gemm_workspace / rmsmp_conv_implicit_workspace
 *                           as rmsmp_gemm / rmsmp_conv_implicit, A operand read from d_workspace.
 * Errors: as the plain calls, plus BUFFER_TOO_SMALL; VARIANT when the tensor kernel cannot run
 * the problem (K or Cin not a multiple of 16, ...).
 */
rmsmp_status rmsmp_workspace_bytes(const rmsmp_layer* layer, size_t* bytes);
rmsmp_status rmsmp_expand_weights(const rmsmp_layer* layer, const void* d_packed, void* d_workspace,
                                  size_t workspace_bytes, void* stream);
rmsmp_status rmsmp_gemm_workspace(const rmsmp_layer* layer, const void* d_packed,
                                  const void* d_workspace, const int8_t* d_act, int64_t N,
                                  int64_t ld_act, float act_step, float* d_out, int64_t ld_out,
                                  rmsmp_out_layout out_layout, int32_t* d_acc, void* stream);
rmsmp_status rmsmp_conv_implicit_workspace(const rmsmp_layer* layer, const void* d_packed,
                                           const void* d_workspace, const int8_t* d_act, int B,
                                           int H, int W, int stride, int pad, float act_step,
                                           float* d_out, rmsmp_out_layout out_layout,
                                           int32_t* d_acc, void* stream);

/*
 * Layer chaining without the fp32 round trip.  The paper runs the quantized model layer by layer
 * with 4-bit activations between layers (Section 3.1, Algorithm 1's forward pass); these calls
 * fuse the NEXT layer's activation quantizer into the epilogue: instead of
 * y[n][m] = float(acc) * (wstep_m * act_step) they write the 4-bit code of that same y,
 *     d_next_codes[n * ld_codes + m] = code(y[n][m]; next_alpha, next_kind),
 * with exactly the arithmetic of rmsmp_quantize_act (RMSMP_ACT_U4 clips at 0, which is the ReLU;
 * RMSMP_ACT_S4 keeps the sign), so the result equals rmsmp_*_workspace followed by
 * rmsmp_quantize_act byte for byte while writing 1 byte per output instead of 4 and saving the
 * quantizer's pass.  [N][M] order only (conv: [B][Ho][Wo][M], ld_codes = M): that is the next
 * layer's input layout.  d_next_codes: device, N * ld_codes bytes; bulk stores are used when it is
 * 16-byte aligned and ld_codes is a multiple of 16.  *h_next_step (host, may be NULL) receives
 * next_alpha/15 or next_alpha/7.  Errors: as rmsmp_*_workspace, plus SCALE for a bad next_alpha;
 * VARIANT when the tensor kernel cannot run the problem.
 */
rmsmp_status rmsmp_gemm_workspace_requant(const rmsmp_layer* layer, const void* d_packed,
                                          const void* d_workspace, const int8_t* d_act, int64_t N,
                                          int64_t ld_act, float act_step, float next_alpha,
                                          rmsmp_act_kind next_kind, int8_t* d_next_codes,
                                          int64_t ld_codes, float* h_next_step, void* stream);
rmsmp_status rmsmp_conv_implicit_workspace_requant(const rmsmp_layer* layer, const void* d_packed,
                                                   const void* d_workspace, const int8_t* d_act,
                                                   int B, int H, int W, int stride, int pad,
                                                   float act_step, float next_alpha,
                                                   rmsmp_act_kind next_kind, int8_t* d_next_codes,
                                                   float* h_next_step, void* stream);

/*
 * Linear layer for callers that cannot allocate device memory (the paper has no counterpart:
 * this is a deployment convenience of the library).  Same computation and same results as
 * rmsmp_expand_weights followed by rmsmp_gemm_workspace, but the scratch for the expanded
 * weights is a fixed 4 MiB array that is part of the loaded library (each GPU that loads the
 * library holds it until the process exits), so the call never allocates or frees anything.
 * Meant for code that runs under a runtime with a fixed memory arena, in a latency-critical
 * loop, or anywhere else cudaMalloc is off limits.
 *   - Limit: layer->M * layer->Kp <= 4 MiB (4,194,304 bytes), else RMSMP_ERR_BUFFER_TOO_SMALL.
 *   - Only the tensor-core kernel is available here: a layer it cannot run (K or ld_act not a
 *     multiple of 16) is refused with RMSMP_ERR_VARIANT instead of falling back to CUDA cores.
 *   - The first call on each device looks up the array's device address
 *     (cudaGetSymbolAddress); with lazy module loading that lookup is also the moment the driver
 *     places the array (and this library's kernels) on the device.  Make that first call during
 *     set-up, outside any stream capture and before the memory budget is frozen.
 *   - All calls share the one array, and it keeps what the last call wrote.  Each call rewrites
 *     every byte it later reads, so stale contents are harmless, but two calls whose GPU work
 *     overlaps (different streams, or different host threads) race on it: serialise them.
 *   - Every argument is checked before anything is queued: a refused call leaves the array, and
 *     any earlier call still running on it, untouched.
 * Arguments and other errors: as rmsmp_gemm (NULL, BAD_LAYER, SHAPE, SCALE, ALIGN, ARCH, CUDA).
 */
rmsmp_status rmsmp_gemm_builtin_scratch(const rmsmp_layer* layer, const void* d_packed,
                                        const int8_t* d_act, int64_t N, int64_t ld_act,
                                        float act_step, float* d_out, int64_t ld_out,
                                        rmsmp_out_layout out_layout, int32_t* d_acc, void* stream);

/*
 * Read the device status word of a packed buffer (synchronises the stream; the paper, which
 * describes an FPGA datapath, has no counterpart).  Kernels never
 * trap: a bounded wait that runs out stores RMSMP_ERR_TIMEOUT there and the kernel returns.
 */
rmsmp_status rmsmp_last_device_status(const void* d_packed, void* stream);

/*
 * Self-check of the failure path (no counterpart in the paper).  Every wait inside the library's
 * kernels is bounded: when one runs out the kernel gives up, records RMSMP_ERR_TIMEOUT in a status
 * word and returns, so the context stays usable.  This call launches one warp that waits, with that
 * same bounded wait, on a barrier nobody will ever signal; after `limit_cycles` SM clock cycles
 * (1 .. 200,000,000, i.e. at most about a tenth of a second) the wait expires and the kernel stores
 * RMSMP_ERR_TIMEOUT to *d_status_word (4 bytes of device memory, which the caller has zeroed).
 * Asynchronous on `stream`; nothing faults, traps or hangs.  Errors: NULL, SHAPE, ARCH, CUDA.
 */
rmsmp_status rmsmp_selftest_bounded_wait(int64_t limit_cycles, uint32_t* d_status_word, void* stream);

/*
 * Measurement helper (no counterpart in the paper): the tensor-pipe ceiling of the current GPU
 * for the MMA shape the contraction kernel issues (M=128, N=n_cols, operands resident in shared
 * memory, every SM busy, no loads or stores).  use_bf16 = 0 measures kind::i8 (the INT8 roofline
 * the layer kernels are reported against), 1 measures bf16 for calibration.  Runs `iters`
 * k-blocks of 4 instructions per SM, synchronises, writes tera-operations per second
 * (2 ops per multiply-accumulate) to *h_tops and the duration to *h_ms (may be NULL).
 * d_status_word: 4 bytes of device memory the kernel may record a wait time-out in.
 * Errors: NULL, SHAPE (iters outside 1..2^22, n_cols not a multiple of 16 in 16..256), ARCH,
 * CUDA, TIMEOUT.
 */
rmsmp_status rmsmp_measure_mma_peak(int use_bf16, int n_cols, int iters, uint32_t* d_status_word,
                                    float* h_tops, float* h_ms, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* RMSMP_H_ */
