/*
 * bro_ref — CPU oracle for the block-rotated MXFP4 W4A4 linear layer.
 *
 * TEST INFRASTRUCTURE ONLY.  This is a plain, slow, obviously-correct restatement of what the
 * method computes, written from the paper's text.  It shares no code, header, table or helper
 * with the CUDA library; only the tests, the smoke check and the benchmark's CPU-baseline leg
 * may call it.  The product path never routes through it.
 *
 * What it follows:
 *   - Block-diagonal orthogonal rotation R_block = diag(R_1..R_B), R_i^T R_i = I, block aligned
 *     with the MX group                                         (paper Sec. 4.3, Eq. 1)
 *   - R_i is a Hadamard matrix (Sylvester construction, normalised by 1/sqrt(block)); the
 *     online transform is a fast Hadamard transform             (Sec. 4.3 "Reduced online
 *     computing", Sec. 5.1, Sec. 6)
 *   - MXFP4: E2M1 elements (1 sign, 2 exponent, 1 mantissa bit), groups of 32 that share one
 *     E8M0 power-of-two scale, symmetric                        (Sec. 4.1)
 *   - Scale and rounding rule: the OCP Microscaling rule the paper cites in Sec. 1:
 *     shared exponent = floor(log2(amax)) - emax_elem with emax_elem = 2 for E2M1, elements
 *     rounded to nearest, ties to even, saturating at +-6.
 *   - W4A4 linear: y = Q(x R) . Q(W R)^T                          (Sec. 1, Sec. 4.2, Sec. 4.3)
 *
 * Pin status: every function below is pinned by the CPU tests (orthogonality, norm
 * preservation, exact inversion, closed forms, an independent O(B^2) definition, worked E2M1
 * examples, brute-force nearest-grid search, idempotence, integer-matmul special cases,
 * the per-element error bound).  One exception: bro_ref_group_mse's *qualitative ordering*
 * between rotation sizes (Sec. 5.2, Fig. 6/7) is "parity unpinned" — the paper prints figures,
 * not numbers; the MSE arithmetic itself is pinned against a numpy restatement.  The scale
 * statistics (outlier groups, histograms, inflation counts) are pinned by brute force in numpy,
 * by conservation (every group is counted once) and by a hand-built row with one outlier channel.
 *
 * Data formats (all host pointers):
 *   bf16 input        : uint16_t, the upper 16 bits of the IEEE fp32 pattern.
 *   codes             : uint8_t [rows, K/2]; byte j of a row holds element 2j in bits 0..3 and
 *                       element 2j+1 in bits 4..7; a code is sign<<3 | mag, mag 0..7 <->
 *                       {0, .5, 1, 1.5, 2, 3, 4, 6}.
 *   scales            : uint8_t [rows, K/32], row-major; byte = E + 127, value 2^E.
 * All functions return 0 on success, non-zero on a bad argument.
 */
#ifndef BRO_REF_H
#define BRO_REF_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Number of OpenMP threads the oracle will use (1 if built without OpenMP). */
int bro_ref_num_threads(void);
void bro_ref_set_num_threads(int n);

/* The fp32 constant c_B = nearest fp32 to 1/sqrt(block) used to normalise H_B. */
float bro_ref_hadamard_norm(int64_t block);

/* Rotation only (Eq. 1 with Hadamard R_i): y[m, :] = x[m, :] R_block, fp32 out [M, K] dense.
 * block in {2^k}; block == 0 means block = K (global rotation, K must be a power of two). */
int bro_ref_rotate(const uint16_t* x_bf16, int64_t M, int64_t K, int64_t ldx, int block,
                   float* y);

/* Randomised block rotation (Sec. 5.1: "block-wise randomized Hadamard rotations"; the random
 * Hadamard construction of the rotation methods the paper builds on): R_i = diag(s) H / sqrt(block)
 * with s a vector of +-1 over the K channels, so y[m, :] = (x[m, :] * s) R_block.  signs_bf16 holds
 * one bf16 value per channel whose SIGN BIT is s (the magnitude is ignored); NULL means all +1.
 * The random draw itself is an input: the oracle consumes no random numbers. */
int bro_ref_rotate_rs(const uint16_t* x_bf16, int64_t M, int64_t K, int64_t ldx, int block,
                      const uint16_t* signs_bf16, float* y);

/* MXFP4 quantisation of fp32 rows (Sec. 4.1): per group of 32, E8M0 scale + 32 E2M1 codes. */
int bro_ref_quantize(const float* y, int64_t rows, int64_t K, uint8_t* codes, uint8_t* scales);

/* Decode codes+scales to fp64 values [rows, K] (exact). */
int bro_ref_decode(const uint8_t* codes, const uint8_t* scales, int64_t rows, int64_t K,
                   double* out);

/* Activation path: rotate then quantise. */
int bro_ref_rotate_quantize_mxfp4(const uint16_t* x_bf16, int64_t M, int64_t K, int64_t ldx,
                                  int block, uint8_t* codes, uint8_t* scales);

/* Activation path with the randomised rotation (signs_bf16 as in bro_ref_rotate_rs). */
int bro_ref_rotate_quantize_mxfp4_rs(const uint16_t* x_bf16, int64_t M, int64_t K, int64_t ldx,
                                     int block, const uint16_t* signs_bf16, uint8_t* codes,
                                     uint8_t* scales);

/* Weight path: identical arithmetic applied to the rows of W[N, K] (offline). */
int bro_ref_pack_weights(const uint16_t* w_bf16, int64_t N, int64_t K, int64_t ldw, int block,
                         uint8_t* wcodes, uint8_t* wscales);

/* y[m,n] = sum_k deq_a[m,k] * deq_w[n,k] in fp64, index order; S[m,n] = sum_k |deq_a*deq_w|.
 * S may be NULL. */
int bro_ref_gemm_mxfp4(const uint8_t* acodes, const uint8_t* ascales, const uint8_t* wcodes,
                       const uint8_t* wscales, int64_t M, int64_t N, int64_t K, double* y,
                       double* S);

/* The same sums for a list of (m, n) points only — for sampled parity at large sizes. */
int bro_ref_gemm_mxfp4_points(const uint8_t* acodes, const uint8_t* ascales,
                              const uint8_t* wcodes, const uint8_t* wscales, int64_t M,
                              int64_t N, int64_t K, const int64_t* pm, const int64_t* pn,
                              int64_t npoints, double* y, double* S);

/* Whole layer: rotate+quantise x, then the GEMM against packed weights. */
int bro_ref_linear(const uint16_t* x_bf16, int64_t M, int64_t K, int64_t ldx, int block,
                   const uint8_t* wcodes, const uint8_t* wscales, int64_t N, double* y,
                   double* S);

/* Per-group quantisation error: mse[r, g] = mean_{i in group} (y[r,i] - deq[r,i])^2, fp64. */
int bro_ref_group_mse(const float* y, const uint8_t* codes, const uint8_t* scales,
                      int64_t rows, int64_t K, double* mse);

/* The 4-bit formats the paper compares MXFP4 with (Sec. 3.1, Sec. 3.2 / Fig. 2, Sec. 4.1 / Fig. 3),
 * all symmetric, group of 32, applied to fp32 rows y:
 *   0 MXFP4   E2M1 elements, E8M0 scale 2^E, E = floor(log2 amax) - 2           (as bro_ref_quantize)
 *   1 BFP4    E2M1 elements, FP16 scale s = fp16(amax / 6)                       ("FP4 variant of BINT4")
 *   2 MXINT4  INT4 elements k/4, k in [-7, 7], E8M0 scale 2^E, E = floor(log2 amax)
 *   3 BINT4   INT4 elements k in [-7, 7], FP16 scale s = fp16(amax / 7)          (RTN, block 32, FP16 scale)
 * and INT4 with one scale per ROW of y instead of per group (Sec. 3.2 / Fig. 2: per-channel symmetric
 * for weights, per-token asymmetric for activations):
 *   4 INT4 row, symmetric    k in [-7, 7], s = fp16(amax_row / 7)
 *   5 INT4 row, asymmetric   codes q in [0, 15] over the range [lo, hi] = [min(row, 0), max(row, 0)]:
 *                            s = fp16((hi - lo) / 15), zero point z = rint(-lo / s) (clamped to 15),
 *                            q = clamp(rint(y / s) + z, 0, 15), dequantised (q - z) s
 * The paper names the formats but gives no formulas; the scale and rounding rules above are this
 * build's reading (round to nearest even everywhere, saturating; fp16 scale = the fp32 quotient
 * rounded to nearest-even fp16, clamped to the largest finite fp16; a zero scale gives all zeros).
 * Writes the dequantised values (exact in fp64) to deq[rows, K]. */
int bro_ref_fake_quantize(const float* y, int64_t rows, int64_t K, int format, double* deq);

/* ---- scale statistics behind the regular-block / outlier-block analysis --------------------------
 * (Sec. 4.1: blocks are "regular" if they hold no outlier and "outlier blocks" otherwise; Sec. 4.2,
 * Fig. 6 caption: outliers are the top 0.1 % of the activations by absolute value; App. A.3: most
 * regular blocks' scales grow under global rotation, block rotation removes most of that growth.)
 * The "scale" here is the E8M0 byte the MXFP4 quantiser assigns to a group of 32 (bro_ref_quantize);
 * the scales "before rotation" are those of the rotation with block = 1, which is the identity.
 *
 * Outlier groups: with n = M*K entries and k = ceil(n * top_ppm / 1e6) (at least 1), t = the k-th
 * largest |x|; an entry is an outlier iff |x| >= t (ties at t all count); mask[m, g] = 1 iff group g of
 * row m holds an outlier.  *threshold_bits receives the bf16 pattern of t. */
int bro_ref_outlier_groups(const uint16_t* x_bf16, int64_t M, int64_t K, int64_t ldx, int64_t top_ppm,
                           uint8_t* mask, uint16_t* threshold_bits);

/* hist[c][b] = number of groups of class c (0 regular, 1 outlier, by mask) whose scale byte is b. */
int bro_ref_scale_histogram(const uint8_t* scales, const uint8_t* mask, int64_t n_groups,
                            uint64_t* hist /* [2][256] */);

/* counts[c][j]: groups of class c whose scale byte after the rotation is lower (j = 0), equal (1) or
 * higher (2) than before it. */
int bro_ref_scale_inflation(const uint8_t* scales_before, const uint8_t* scales_after,
                            const uint8_t* mask, int64_t n_groups, uint64_t* counts /* [2][3] */);

/* ---- the producer of the online-rotated activations -----------------------------------------------
 * The one rotation paid at inference sits directly before down_proj (Sec. 4.3 "Reduced online
 * computing"; Sec. 6), whose input in the LLaMA-family models the paper evaluates is the gated MLP
 * activation h = silu(gate) * up.  The paper does not spell that producer out; this build's reading, in
 * fp32 with every operation one IEEE round-to-nearest step so that two implementations agree bit for bit:
 *   t = -|g|;  e = exp(t) as  n = rint(t * log2e), r = fma(n, -ln2_hi, t), r = fma(n, -ln2_lo, r),
 *   p = 1 + r (1 + r (1/2 + r (1/6 + r (1/24 + r (1/120 + r / 720))))) by Horner with fma, e = p * 2^n
 *   (e = 0 for t < -86);  sigmoid = (g >= 0 ? 1 : e) / (1 + e);  h = bf16_rne((g * sigmoid) * u).
 * Pinned against the exact function (|error| of the fp32 value <= 4e-7 relative + 4e-36 |u|), special values,
 * and an independent bf16 rounding (torch). */
int bro_ref_swiglu_f32(const uint16_t* gate_bf16, const uint16_t* up_bf16, int64_t n, float* h32);
int bro_ref_swiglu(const uint16_t* gate_bf16, const uint16_t* up_bf16, int64_t M, int64_t K, int64_t ldg,
                   int64_t ldu, uint16_t* h_bf16 /* [M, K] dense */);
/* h as above, then the activation path (rotate + MXFP4 quantise) on it. */
int bro_ref_swiglu_rotate_quantize_mxfp4(const uint16_t* gate_bf16, const uint16_t* up_bf16, int64_t M,
                                         int64_t K, int64_t ldg, int64_t ldu, int block,
                                         const uint16_t* signs_bf16, uint8_t* codes, uint8_t* scales);

#ifdef __cplusplus
}
#endif
#endif /* BRO_REF_H */
