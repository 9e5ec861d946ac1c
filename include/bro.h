/*
 * bro.h — C ABI of libbro: the W4A4 MXFP4 linear layer with block-Hadamard rotation on one
 * NVIDIA B200 (sm_100a).
 *
 * The operations follow "Block Rotation is All You Need for MXFP4 Quantization"
 * (arXiv 2511.04214):
 *   - rotation   x -> x R_block, R_block = diag(R_1..R_B) with orthogonal blocks aligned with
 *                the MX group (Sec. 4.3, Eq. 1); R_i = H_block / sqrt(block), H the Sylvester
 *                Hadamard matrix, applied as a fast transform (Sec. 4.3 "Reduced online
 *                computing", Sec. 5.1);
 *   - MXFP4      E2M1 elements, groups of 32 sharing one E8M0 power-of-two scale (Sec. 4.1),
 *                scale exponent = floor(log2 amax) - 2, round-to-nearest-even, saturate at +-6
 *                (the OCP Microscaling rule the paper cites in Sec. 1);
 *   - W4A4       y = Q(x R) Q(W R)^T with fp32 accumulation (Sec. 1, Sec. 4.2).
 *
 * Conventions
 *   - Unless a parameter says "host", every pointer is a DEVICE pointer owned by the caller.
 *     The library allocates no device memory.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls
 *     enqueue work and return without synchronising.  The returned status covers argument
 *     validation and launch errors only.
 *   - Every device-side wait is bounded by a time budget (two seconds on the device's own
 *     nanosecond timer).  If one expires (which indicates a bug or a broken device, never a data
 *     condition) the kernel records BRO_ERR_TIMEOUT and the place of the wait in a device-side
 *     status word and returns; bro_last_device_status() reads and clears that word.  There is ONE
 *     status word per device, shared by all streams and all calls on that device (it lives in the
 *     library's device image, not in a caller buffer, so that entry points without a workspace
 *     can report too): it says that some kernel since the last read gave up, not which call.
 *   - The library keeps no other state that affects results: which kernel variant runs is a
 *     function of the arguments alone (the *_ex entry points take explicit flags; nothing is
 *     read from the environment).  One-time per-device set-up (kernel attributes) is
 *     thread-safe.
 *   - No exception crosses this boundary.  Invalid arguments return an error code; they never
 *     lead to undefined behaviour.  M == 0 or N == 0 returns BRO_OK without a launch.
 *   - bf16 tensors are row-major with a leading dimension in ELEMENTS.
 *
 * Data formats
 *   codes   uint8 [rows, K/2], row-major, dense.  Byte j of a row holds element 2j in bits 0..3
 *           and element 2j+1 in bits 4..7.  A code is sign<<3 | mag, mag 0..7 <->
 *           {0, 0.5, 1, 1.5, 2, 3, 4, 6}.  The sign bit of a value that rounds to zero is kept.
 *   scales  uint8, one per (row, group of 32): byte = E + 127 for the scale 2^E.  0xFF is never
 *           produced for finite input.
 *           BRO_LAYOUT_CANONICAL: [rows, K/32] row-major.
 *           BRO_LAYOUT_GEMM: the order the tensor core reads.  Rows are padded to a multiple of
 *           128 and K to a multiple of 256; the buffer is an array [ceil(rows/128)][KB] of
 *           512-byte blocks, KB = 2*ceil(K/256), block (i, j) covering rows 128i..128i+127 and
 *           groups 4j..4j+3; inside a block the byte for (row r, group g) sits at
 *           (r%32)*16 + ((r%128)/32)*4 + (g%4).  Padding bytes are written as 0.
 *           bro_scale_offset() returns the byte offset of one (row, group) in either layout.
 */
#ifndef BRO_H
#define BRO_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  BRO_OK = 0,
  BRO_ERR_NULL = 1,        /* a required pointer is NULL */
  BRO_ERR_SHAPE = 2,       /* a size, leading dimension or block value is not allowed */
  BRO_ERR_ALIGN = 3,       /* a pointer or leading dimension is not aligned as required */
  BRO_ERR_UNSUPPORTED = 4, /* valid request that this build does not implement */
  BRO_ERR_WORKSPACE = 5,   /* workspace too small */
  BRO_ERR_CUDA = 6,        /* a CUDA runtime/driver call failed */
  BRO_ERR_TIMEOUT = 7,     /* a bounded device-side wait expired */
  BRO_ERR_ARCH = 8         /* the current device is not compute capability 10.x */
} bro_status;

typedef enum { BRO_LAYOUT_CANONICAL = 0, BRO_LAYOUT_GEMM = 1 } bro_layout;
typedef enum { BRO_OUT_BF16 = 0, BRO_OUT_F32 = 1 } bro_out_dtype;
/* 4-bit formats of the analysis entry point (see bro_group_quant_error_fmt). */
typedef enum {
  BRO_FMT_MXFP4 = 0, BRO_FMT_BFP4 = 1, BRO_FMT_MXINT4 = 2, BRO_FMT_BINT4 = 3,
  /* bro_rotate_fake_quantize(_ws) only: INT4 with one scale per row, and no quantisation at all */
  BRO_FMT_INT4_ROW_SYM = 4, BRO_FMT_INT4_ROW_ASYM = 5, BRO_FMT_NONE = 6
} bro_format;

/* Human-readable name of a status code (static string, never NULL). */
const char* bro_status_string(bro_status s);

/* Text of the most recent CUDA runtime/driver error this thread saw inside a libbro call that
 * returned BRO_ERR_CUDA ("" if none).  Static storage; valid until the next libbro call. */
const char* bro_last_cuda_error(void);

/* rows*K/2: bytes of a packed code tensor. */
size_t bro_codes_bytes(int64_t rows, int64_t K);
/* Bytes of a scale tensor in the given layout (padded for BRO_LAYOUT_GEMM). 0 on bad input. */
size_t bro_scales_bytes(int64_t rows, int64_t K, bro_layout layout);
/* Byte offset of the scale of (row, group) inside a scale tensor of `rows` x K. */
size_t bro_scale_offset(int64_t row, int64_t group, int64_t rows, int64_t K, bro_layout layout);
/* Workspace bro_gemm_mxfp4 needs for this problem (may be 0). */
size_t bro_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K);
/* Workspace bro_linear needs: quantised activations (codes + GEMM-layout scales) + the GEMM's. */
size_t bro_linear_workspace_bytes(int64_t M, int64_t N, int64_t K);

/* Synchronises `stream`, then returns and clears the device-side status word of the current
 * device: BRO_OK, or BRO_ERR_TIMEOUT if a kernel gave up on a bounded wait since the last call.
 * BRO_ERR_CUDA if the synchronisation itself reports an error. */
bro_status bro_last_device_status(void* stream);
/* The same, and *site (if not NULL) receives the number of the wait that expired (0 if none):
 * 1-3 rotate+quantize ring (full / empty / drain), 4-9 GEMM (operands full / stage empty /
 * accumulator full / accumulator free / drain / tensor memory), 10 the self-test below. */
bro_status bro_last_device_status_ex(void* stream, int* site);

/*
 * Online activation path (Sec. 4.3 Eq. 1 + Sec. 4.1): for every row of x[M, K] (bf16) and every
 * aligned block of `block` channels, y = (H_block x) / sqrt(block) in fp32 — butterflies in
 * ascending stride order, one multiply by the fp32 nearest 1/sqrt(block) at the end — then each
 * group of 32 values of y is quantised to MXFP4.
 *   block   32, 64 or 128; or 0 for block = K (global rotation; K must then be a power of two,
 *           32 <= K <= 32768); or 2, 4, 8, 16 — a rotation inside the MX group (Sec. 5.2 sweeps the
 *           rotation dimension below as well as above the group size; the butterfly stops early).
 *   ldx     row stride of x in elements, >= K, multiple of 8.
 *   codes   out, [M, K/2] bytes, 16-byte aligned.
 *   scales  out, bro_scales_bytes(M, K, layout) bytes, 16-byte aligned.
 * Requirements: K % 32 == 0, K % block == 0, x 16-byte aligned.
 */
bro_status bro_rotate_quantize_mxfp4(const void* x_bf16, int64_t M, int64_t K, int64_t ldx,
                                     int block, void* codes, void* scales, bro_layout layout,
                                     void* stream);

/*
 * Offline weight path: the same arithmetic applied to the rows of w[N, K] (the rotation acts on
 * the K axis of both operands, so (x R)(W R)^T = x W^T before quantisation, Eq. 1).  Scales are
 * written in BRO_LAYOUT_GEMM.
 */
bro_status bro_pack_weights(const void* w_bf16, int64_t N, int64_t K, int64_t ldw, int block,
                            void* wcodes, void* wscales, void* stream);

/*
 * Block-scaled MXFP4 x MXFP4 GEMM (Sec. 1 W4A4; Sec. 4.2):
 *   y[m, n] = sum_g 2^(Ea[m,g] + Ew[n,g]) * sum_{k in group g} a[m,k] * w[n,k]
 * with fp32 accumulation on the tensor cores and the result written as bf16 (round to nearest
 * even) or fp32.
 *   acodes/wcodes    [M, K/2] and [N, K/2] bytes, 128-byte aligned.
 *   ascales/wscales  BRO_LAYOUT_GEMM, 128-byte aligned.
 *   y                [M, ldy] of out_dtype, 16-byte aligned; ldy >= N, ldy*sizeof(elem) % 16 == 0.
 *   workspace        bro_gemm_workspace_bytes(M, N, K) bytes (may be NULL when that is 0).
 * Requirements: K % 32 == 0.
 */
bro_status bro_gemm_mxfp4(const void* acodes, const void* ascales, const void* wcodes,
                          const void* wscales, int64_t M, int64_t N, int64_t K, void* y,
                          int64_t ldy, bro_out_dtype out_dtype, void* workspace,
                          size_t workspace_bytes, void* stream);

/*
 * The whole layer on one stream: bro_rotate_quantize_mxfp4(x) into the workspace, then
 * bro_gemm_mxfp4 against weights packed by bro_pack_weights with the same `block`.
 *   workspace   bro_linear_workspace_bytes(M, N, K) bytes, 1024-byte aligned.
 *   y_bf16      [M, ldy] bf16.
 */
bro_status bro_linear(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int block,
                      const void* wcodes, const void* wscales, int64_t N, void* y_bf16,
                      int64_t ldy, void* workspace, size_t workspace_bytes, void* stream);

/*
 * The rotation fused into its producer.  The one rotation paid at inference sits before down_proj
 * (Sec. 4.3, "Reduced online computing"; Sec. 6), whose input in the LLaMA-family models the paper
 * evaluates is the gated activation h = silu(gate) * up.  These entry points compute h inside the
 * rotate+quantize kernel, so h is never written to or read from device memory:
 *   h[m, k] = bf16_rne( (g * sigmoid(g)) * u ),  g = gate[m, k], u = up[m, k]  (bf16 in, fp32 arithmetic)
 * with sigmoid from a fixed sequence of IEEE fp32 operations — e = exp(-|g|) by n = rint(-|g| log2e), two
 * fused multiply-adds of range reduction, a degree-6 Horner polynomial and an exact scaling by 2^n; e = 0
 * below -86; sigmoid = (g >= 0 ? 1 : e) / (1 + e) — accurate to a few fp32 ulps and bit-reproducible (the
 * paper does not spell the producer out; this is the library's reading).  Then the activation path of
 * bro_rotate_quantize_mxfp4 on h.
 *   gate_bf16, up_bf16  [M, K] bf16, row strides ldg / ldu in elements (>= K, multiples of 8), 16-byte aligned.
 *   block               2, 4, 8, 16, 32, 64 or 128 (block = 0 is not offered here: BRO_ERR_UNSUPPORTED).
 *   signs_bf16          NULL or the +-1 vector of the randomised rotation.
 * bro_swiglu_bf16 is the producer alone (h as a bf16 tensor [M, ldh]), for callers that need h itself.
 * bro_swiglu_linear is bro_linear(_rs) with the fused producer in front: y = Q(h R) Q(W R)^T.
 */
bro_status bro_swiglu_rotate_quantize_mxfp4(const void* gate_bf16, const void* up_bf16, int64_t M, int64_t K,
                                            int64_t ldg, int64_t ldu, int block, const void* signs_bf16,
                                            void* codes, void* scales, bro_layout layout, void* stream);
bro_status bro_swiglu_bf16(const void* gate_bf16, const void* up_bf16, int64_t M, int64_t K, int64_t ldg,
                           int64_t ldu, void* h_bf16, int64_t ldh, void* stream);
bro_status bro_swiglu_linear(const void* gate_bf16, const void* up_bf16, int64_t M, int64_t K, int64_t ldg,
                             int64_t ldu, int block, const void* signs_bf16, const void* wcodes,
                             const void* wscales, int64_t N, void* y_bf16, int64_t ldy, void* workspace,
                             size_t workspace_bytes, void* stream);

/*
 * Packed weights with a descriptor.  bro_pack_weights writes two bare buffers; nothing in them says
 * which rotation they were packed with, so bro_linear cannot notice weights packed with another block
 * size or sign vector (the rotation would no longer cancel, Eq. 1, and the layer would silently
 * compute something else).  A caller who wants that check keeps this HOST-side descriptor with the
 * buffers (and stores it as the header of a weight file): bro_pack_weights_desc fills it,
 * bro_linear_packed refuses (BRO_ERR_SHAPE) activations whose K, block or use of a sign vector differ,
 * and a descriptor with the wrong magic or layout version (BRO_ERR_UNSUPPORTED).
 *   signs_bf16  NULL for the plain rotation, else the +-1 vector (see the randomised forms below).
 * All other arguments, requirements and errors are those of bro_pack_weights(_rs) / bro_linear(_rs).
 */
#define BRO_WEIGHTS_MAGIC 0x344F5242u /* "BRO4" */
#define BRO_WEIGHTS_VERSION 1u        /* codes row-major [N, K/2]; scales in BRO_LAYOUT_GEMM */
typedef struct {
  uint32_t magic;     /* BRO_WEIGHTS_MAGIC */
  uint32_t version;   /* BRO_WEIGHTS_VERSION */
  int64_t N, K;
  int32_t block;      /* rotation block the weights were packed with: 2 .. 128 or 0 (= K) */
  int32_t randomised; /* 1 if a sign vector was applied */
  const void* codes;  /* device, bro_codes_bytes(N, K) bytes */
  const void* scales; /* device, bro_scales_bytes(N, K, BRO_LAYOUT_GEMM) bytes */
} bro_packed_weights;
bro_status bro_pack_weights_desc(const void* w_bf16, int64_t N, int64_t K, int64_t ldw, int block,
                                 const void* signs_bf16, void* wcodes, void* wscales,
                                 bro_packed_weights* desc /* host, out */, void* stream);
bro_status bro_linear_packed(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int block,
                             const void* signs_bf16, const bro_packed_weights* weights /* host */,
                             void* y_bf16, int64_t ldy, void* workspace, size_t workspace_bytes,
                             void* stream);

/*
 * Randomised block rotation (Sec. 5.1, "block-wise randomized Hadamard rotations"): the same three
 * operations with R_i = diag(s) H_block / sqrt(block), s a vector of +-1 over the K channels, i.e.
 * channel k of every row is multiplied by s_k (exactly, a sign-bit flip) before the transform.
 *   signs_bf16  device, [K] bf16, 16-byte aligned; only the SIGN BIT of each value is used
 *               (+1 / -1).  The caller draws it; the library consumes no random numbers.
 * Activations and weights must use the same sign vector, so that (x R)(W R)^T = x W^T.
 * All other arguments and requirements are those of the plain entry points.
 */
bro_status bro_rotate_quantize_mxfp4_rs(const void* x_bf16, int64_t M, int64_t K, int64_t ldx,
                                        int block, const void* signs_bf16, void* codes,
                                        void* scales, bro_layout layout, void* stream);
bro_status bro_pack_weights_rs(const void* w_bf16, int64_t N, int64_t K, int64_t ldw, int block,
                               const void* signs_bf16, void* wcodes, void* wscales, void* stream);
bro_status bro_linear_rs(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int block,
                         const void* signs_bf16, const void* wcodes, const void* wscales, int64_t N,
                         void* y_bf16, int64_t ldy, void* workspace, size_t workspace_bytes,
                         void* stream);

/*
 * Analysis: the quantisation error the rotation leaves per MX group (Sec. 4.1-4.2 and Fig. 3 / 6:
 * error of regular vs. outlier blocks under the shared power-of-two scale; App. A.3).  For every
 * row of x and every group of 32 channels of y = x R_block:
 *   mse[m, g] = mean_i (y_i - deq(Q(y))_i)^2
 * with Q the MXFP4 quantiser of bro_rotate_quantize_mxfp4.  Nothing else is written.
 *   block       2, 4, 8, 16, 32, 64, 128 or 0 (= K), as above; also 1 (no rotation);
 *   signs_bf16  NULL or the +-1 vector of the randomised rotation;  mse  device, fp32 [M, K/32], dense.
 * Arithmetic: differences are exact, squares and their sum are rounded in fp32 (relative error of a
 * few 2^-24 against an fp64 evaluation).
 */
bro_status bro_group_quant_error(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int block,
                                 const void* signs_bf16, float* mse, void* stream);

/*
 * The same statistic for the 4-bit formats the paper compares MXFP4 with (Sec. 3.1 BINT4 baseline;
 * Sec. 3.2 / Fig. 2 format study; Sec. 4.1 / Fig. 3 MXFP4 against BFP4), all symmetric with groups
 * of 32 and round to nearest even, saturating:
 *   BRO_FMT_MXFP4   E2M1 elements, scale 2^E, E = floor(log2 amax) - 2
 *   BRO_FMT_BFP4    E2M1 elements, FP16 scale fp16(amax / 6)
 *   BRO_FMT_MXINT4  elements k/4 with |k| <= 7, scale 2^E, E = floor(log2 amax)
 *   BRO_FMT_BINT4   integer elements |k| <= 7, FP16 scale fp16(amax / 7)
 * (the paper names these formats without formulas; the rules above are this library's reading).
 * Only MXFP4 has a GEMM here — the other formats exist for the error analysis.
 */
bro_status bro_group_quant_error_fmt(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int block,
                                     const void* signs_bf16, bro_format format, float* mse,
                                     void* stream);

/*
 * Simulated ("fake") quantisation: rotate, quantise, dequantise.  The paper evaluates every method by
 * simulating the MX formats rather than running a native FP4 GEMM (Sec. 3.1, experimental setup), and
 * its format study compares MXFP4 with BFP4, MXINT4 and BINT4 on the same tensors (Sec. 3.2 / Fig. 2,
 * Sec. 4.1 / Fig. 3); this call produces those tensors.  For every row of x:
 *   deq[m, :] = dequantised values of Q_format((x diag(s) R_block)[m, :]),  fp32, in the ROTATED domain
 * with the quantisers listed above (decisions as in bro_group_quant_error_fmt).  Every value is a 3-bit
 * element times a power of two or an fp16 scale, hence exact in fp32; a negative input that quantises
 * to zero gives -0.0, a group whose fp16 scale rounds to zero gives +0.0 throughout.
 *   block       1 (no rotation), 2, 4, 8, 16 (inside the MX group), 32, 64, 128 or 0 (= K, K a power
 *               of two in [32, 32768])
 *   signs_bf16  NULL or the +-1 vector of the randomised rotation (device, [K] bf16, 16-byte aligned)
 *   deq         device, fp32 [M, K] with row stride ldd >= K elements (ldd % 4 == 0, 16-byte aligned);
 *               columns K .. ldd-1 are not written
 * Errors as for bro_group_quant_error_fmt; M == 0 returns BRO_OK without a launch.  Only MXFP4 has a
 * GEMM in this library: a simulated W4A4 layer in another format is deq_a deq_w^T in the caller's
 * precision.
 */
bro_status bro_rotate_fake_quantize(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int block,
                                    const void* signs_bf16, bro_format format, float* deq, int64_t ldd,
                                    void* stream);
/*
 * The same with a workspace.  Three more values of `format` exist for these two calls (BRO_FMT_NONE
 * needs no workspace and is accepted by both; the per-row formats need one):
 *   BRO_FMT_INT4_ROW_SYM   INT4 with one scale per ROW, symmetric: |k| <= 7, scale fp16(amax_row / 7)
 *   BRO_FMT_INT4_ROW_ASYM  INT4 with one scale per row, asymmetric: codes q in [0, 15] over the range
 *                          [lo, hi] = [min(row, 0), max(row, 0)], scale s = fp16((hi - lo) / 15), zero
 *                          point z = rint(-lo / s) (at most 15), q = clamp(rint(y / s) + z, 0, 15),
 *                          dequantised (q - z) s (+0.0 where q == z)
 *   BRO_FMT_NONE           no quantisation: deq = x diag(s) R_block itself, the fp32 values every other
 *                          format is an approximation of (so that the caller can form any error statistic)
 * The first two are the fifth format of the paper's study (Sec. 3.2 / Fig. 2: "INT4" = per-channel
 * symmetric weights — a row of W is an output channel — and per-token asymmetric activations — a row
 * of X is a token); the paper gives no formulas, the rules above are this library's reading.  They
 * take two passes over x (the first leaves each row's range in the workspace) and need
 *   workspace   device, bro_fake_quantize_workspace_bytes(M, format) bytes (8 per row; 0 for the other
 *               formats, which ignore it), 8-byte aligned; contents undefined afterwards.
 * BRO_ERR_WORKSPACE if it is missing or too small.  bro_rotate_fake_quantize is this call without a
 * workspace.  Everything else as above.
 */
size_t bro_fake_quantize_workspace_bytes(int64_t M, bro_format format);
bro_status bro_rotate_fake_quantize_ws(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int block,
                                       const void* signs_bf16, bro_format format, float* deq, int64_t ldd,
                                       void* workspace, size_t workspace_bytes, void* stream);

/*
 * Scale statistics behind the paper's regular-block / outlier-block argument (Sec. 4.1: "regular
 * blocks" hold no outlier, "outlier blocks" one or more; Sec. 4.2, Fig. 6 caption: outliers are the
 * top 0.1 % of the activations by absolute value; App. A.3, Fig. 8-9: under global rotation the scales
 * of most regular blocks grow, block rotation removes most of that growth).  The "scale" of a group is
 * the E8M0 byte the MXFP4 quantiser gives it.  All results are integers and exact.
 *
 * bro_group_scale_bytes: scales[m, g] (uint8 [M, K/32], dense) = the scale byte of group g of row m of
 *   x R_block.  block = 1 is the identity rotation — the activations as they are ("before rotation");
 *   2, 4, 8, 16 rotate inside the MX group; 32, 64, 128 and 0 (= K) as in bro_rotate_quantize_mxfp4;
 *   signs_bf16 NULL or the +-1 vector.
 *   Nothing else is written.
 */
bro_status bro_group_scale_bytes(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int block,
                                 const void* signs_bf16, uint8_t* scales, void* stream);
/*
 * bro_outlier_groups: with n = M*K entries and k = ceil(n * top_ppm / 1e6) (at least 1; 1000 ppm is the
 *   paper's 0.1 %), t = the k-th largest |x|; an entry is an outlier iff |x| >= t (ties at t all count).
 *   mask[m, g] (uint8 [M, K/32]) = 1 iff group g of row m holds an outlier, else 0.
 *   info       device, 4 x uint32, 16-byte aligned: [0] = the bf16 pattern of t, [1] = 0, [2..3] = k.
 *   workspace  device, bro_outlier_workspace_bytes() bytes, 16-byte aligned (a histogram of the 32768
 *              bf16 magnitudes; overwritten).
 *   Inputs must be finite.
 */
size_t bro_outlier_workspace_bytes(void);
bro_status bro_outlier_groups(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int64_t top_ppm,
                              uint8_t* mask, uint32_t* info, void* workspace, size_t workspace_bytes,
                              void* stream);
/*
 * bro_scale_histogram: hist (device, uint64 [2][256]) is overwritten with the number of groups of each
 *   class (row 0 regular, row 1 outlier, by mask) that have each scale byte.
 * bro_scale_inflation: counts (device, uint64 [2][3]) is overwritten with, per class, the number of
 *   groups whose scale byte after a rotation is lower / equal / higher than before it — counts[0][2]
 *   over the number of regular groups is the "fraction of regular blocks whose scale grows".
 *   scales*, mask: device uint8 [n_groups].
 */
bro_status bro_scale_histogram(const uint8_t* scales, const uint8_t* mask, int64_t n_groups,
                               uint64_t* hist, void* stream);
bro_status bro_scale_inflation(const uint8_t* scales_before, const uint8_t* scales_after,
                               const uint8_t* mask, int64_t n_groups, uint64_t* counts, void* stream);

/*
 * ---- tuning and testing -------------------------------------------------------------------------
 * The *_ex entry points are the plain ones plus a `flags` word that forces a kernel variant the
 * library would not pick by itself for this problem (the plain entry points pass 0).  Every variant
 * computes the same function: codes and scales are bit-identical, GEMM results agree within the
 * accumulation-order tolerance.  They exist so that each variant can be tested and timed on any
 * shape; `signs_bf16` may be NULL (plain rotation) or the +-1 vector of the randomised rotation.
 */
#define BRO_FLAG_RQ_TMA_RING 0x1u     /* rotate+quantize: shared-memory ring fed by TMA (block 32/64/128) */
#define BRO_FLAG_RQ_DIRECT 0x2u       /* rotate+quantize: register-streaming kernel (block 32/64/128) */
#define BRO_FLAG_GEMM_PAIR 0x10u      /* GEMM: two CTAs per 256 x 256 tile (cta_group::2) */
#define BRO_FLAG_GEMM_TILE_N128 0x20u /* GEMM: 128 x 128 tiles */
#define BRO_FLAG_GEMM_TILE_N256 0x40u /* GEMM: 128 x 256 tiles even when N <= 128 */
#define BRO_FLAG_GEMM_NO_SPLIT 0x80u  /* GEMM: no half-width units in the last round of the grid */
#define BRO_FLAG_GEMM_SINGLE 0x100u   /* GEMM: one CTA per 128 x 256 (or 128 x 128) tile, whatever the size */
bro_status bro_rotate_quantize_mxfp4_ex(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int block,
                                        const void* signs_bf16, void* codes, void* scales,
                                        bro_layout layout, uint32_t flags, void* stream);
bro_status bro_gemm_mxfp4_ex(const void* acodes, const void* ascales, const void* wcodes,
                             const void* wscales, int64_t M, int64_t N, int64_t K, void* y, int64_t ldy,
                             bro_out_dtype out_dtype, void* workspace, size_t workspace_bytes,
                             uint32_t flags, void* stream);
bro_status bro_linear_ex(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int block,
                         const void* signs_bf16, const void* wcodes, const void* wscales, int64_t N,
                         void* y_bf16, int64_t ldy, void* workspace, size_t workspace_bytes,
                         uint32_t flags, void* stream);

/*
 * Self-test of the bounded-wait machinery (no counterpart in the paper): launches one warp that
 * waits, with a budget of `budget_ns` nanoseconds (clamped to [1 us, 100 ms]), on a barrier that
 * nothing ever completes.  The wait runs out, the warp records BRO_ERR_TIMEOUT with site 10 in the
 * device status word and the kernel ends normally — nothing faults, and the context stays usable.
 * A following bro_last_device_status() therefore returns BRO_ERR_TIMEOUT once, then BRO_OK.
 */
bro_status bro_selftest_expire_wait(uint64_t budget_ns, void* stream);

/*
 * bro_linear for a caller whose activations and result live in HOST memory (pinned memory gives
 * asynchronous copies).  Copies x_host[M, K] (dense, ldx = K) to the device staging buffer,
 * runs bro_linear, and copies y[M, N] (dense) back to y_host, all on `stream`.
 *   x_stage  device, M*K*2 bytes;  y_stage  device, M*N*2 bytes;  both 16-byte aligned.
 * The call returns after enqueuing; synchronise the stream before reading y_host.
 */
bro_status bro_linear_host(const void* x_host_bf16, int64_t M, int64_t K, int block,
                           const void* wcodes, const void* wscales, int64_t N,
                           void* y_host_bf16, void* x_stage, void* y_stage, void* workspace,
                           size_t workspace_bytes, void* stream);

/*
 * bro_linear for callers that cannot hand over a workspace.  (The paper has no counterpart: this
 * entry point exists for integration reasons only; the arithmetic is bro_linear's.)
 *
 * Who needs it: code that runs where device allocation is off limits — inside a region that is
 * being captured into a CUDA graph by someone else, in a plugin whose host framework owns the
 * allocator and gives the plugin only its input and output tensors, or in a serving loop that
 * has pinned its memory budget and forbids cudaMalloc after start-up.  Such a caller has x, the
 * packed weights and y, but nowhere to put the quantised activations that sit between the two
 * kernels.  Here that intermediate lives in an array compiled into the library:
 *   BRO_STATIC_SCRATCH_BYTES of device memory per GPU, reserved when the library is loaded on
 *   that GPU and held until the process exits, whether or not this function is ever called.
 * The function itself allocates nothing: no cudaMalloc/cudaFree, no allocating library call.
 *
 * Limit: align256(M*K/2) + bro_scales_bytes(M, K, BRO_LAYOUT_GEMM) + bro_gemm_workspace_bytes(M, N, K)
 * must not exceed BRO_STATIC_SCRATCH_BYTES (about M*K <= 31 million elements); a larger
 * problem returns BRO_ERR_WORKSPACE, launches nothing and leaves a one-line explanation in
 * bro_last_cuda_error().  All other arguments, requirements and errors are those of bro_linear.
 *
 * Set-up: the first call on each device looks up the array's device address (the name the
 * host code sees is only a handle, not an address a kernel could use).  Make that first call with
 * the device current and outside any stream capture.  Separately, as for every entry point of
 * this library, the first launch of each kernel variant on a device (one per block size, per
 * size class of the input, per GEMM tile width and output type) loads that kernel and opts it in
 * to its shared-memory size: run one call of every (block, shape class) you will use before
 * capturing.  With block = 0 the call also enqueues a memset of the scale buffer's padding.
 *
 * Sharing: every call on a device uses the same array and finds in it whatever the previous
 * call left.  Each call rewrites everything it later reads (padding included), so stale contents
 * are harmless — but two calls that can run at the same time on one GPU (different streams,
 * different host threads) race on the array.  Keep calls on one stream, or order them yourself.
 */
#define BRO_STATIC_SCRATCH_BYTES ((size_t)16 << 20)
bro_status bro_linear_static(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int block,
                             const void* wcodes, const void* wscales, int64_t N, void* y_bf16,
                             int64_t ldy, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* BRO_H */
