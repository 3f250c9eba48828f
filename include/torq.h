/*
 * torq.h -- C ABI of the B200 (sm_100a) hot path of TORQ's rotated-MXFP4 linear layer.
 *
 * The path is the paper's online inference procedure (Algorithm 3): a token's d features are
 * viewed as d/32 blocks of 32 (step 1), multiplied by the inter-block rotation (step 2) and by
 * the intra-block rotation of each block (step 3), quantized per block to MXFP4 (step 4, Eq. 1)
 * and handed to the next linear layer whose weights already carry the inverse rotation and are
 * themselves MXFP4 (step 5, option B "weight fusion").
 *
 * Conventions for every entry point
 *   - All data pointers are DEVICE pointers owned by the caller; the library allocates nothing
 *     and keeps no reference after the call returns.  `stream` is a cudaStream_t passed as
 *     void* (NULL = the legacy default stream).  Calls only enqueue work; they never synchronise.
 *   - Tokens are rows (row-vector convention): Z = X . R_inter, then per block Z_b . R_intra[b].
 *   - bf16 = bfloat16, u8 = unsigned byte.  Matrices are row-major, densely packed.
 *   - MXFP4 codes: 4 bits per element = sign<<3 | e2m1 magnitude index over
 *     {0, 0.5, 1, 1.5, 2, 3, 4, 6}; two codes per byte, the even element in the low nibble.
 *   - Scales: one E8M0 byte per (row, 32-element block), byte = e + 127 with
 *     e = clamp(floor(log2 amax) - 2, -127, 127) (amax == 0 -> byte 0), stored in the tiled
 *     layout the block-scaled tensor-core instruction reads (see torq_scale_offset).  A scale
 *     buffer always has torq_scales_bytes(rows, k) bytes: rows are padded to a multiple of 128
 *     and K-blocks to a multiple of 4.  Producers in this library write 0x00 (2^-127) into the
 *     padding rows; consumers never let padding reach a stored output.
 *   - R_inter, R_intra, Wq and Ws are constants of the layer.  The tensor-core kernels may start
 *     reading them while the kernel launched just before on the same stream is still finishing
 *     (everything else waits for that kernel), so they must not be written by that kernel: put a
 *     stream synchronisation or any other kernel between producing them and the first call.
 *   - Return value: TORQ_OK or a host-detected error; nothing is launched on error.  Conditions
 *     only the device can see (a bounded wait that ran out) are latched in an error word read by
 *     torq_last_device_error(); a kernel that hits one stops issuing work, drains and returns --
 *     it never traps.  Non-finite inputs are outside the contract (results unspecified, no hang).
 */
#ifndef TORQ_H_
#define TORQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  TORQ_OK = 0,
  TORQ_ERR_NULL = 1,       /* a required pointer is NULL */
  TORQ_ERR_SHAPE = 2,      /* a size violates the stated divisibility / range rules */
  TORQ_ERR_ALIGN = 3,      /* a pointer is not 16-byte aligned */
  TORQ_ERR_ARCH = 4,       /* current device is not compute capability 10.x */
  TORQ_ERR_LAUNCH = 5,     /* CUDA reported an error while encoding descriptors or launching */
  TORQ_ERR_TIMEOUT = 6,    /* (device error word) a bounded wait inside a kernel ran out */
  TORQ_ERR_WORKSPACE = 7   /* workspace missing or smaller than torq_workspace_bytes() */
} torq_status;

typedef enum { TORQ_F32 = 0, TORQ_BF16 = 1 } torq_dtype;

/* Algorithm 3 steps 1-4 (rotation as in Section 5: R = inter then intra; quantizer Eq. 1).
 *   X         [M, d]        bf16
 *   R_inter   [d, d]        bf16, y[m,j] = sum_i x[m,i] R_inter[i,j]; NULL = identity
 *   R_intra   [d/32,32,32]  bf16, z[m,32b+j] = sum_i y[m,32b+i] R_intra[b][i][j]; NULL = identity
 *   out_codes [M, d/2]      u8
 *   out_scales              torq_scales_bytes(M, d) bytes, tiled layout
 * Requires M >= 1, d >= 32, d % 32 == 0, 16-byte aligned pointers.  Accumulation is fp32
 * (inter: tensor cores with exact bf16 products; intra: fp32 FMAs in index order).
 * When R_inter is NULL the call runs the quantize-only kernel (plus the intra step if given). */
torq_status torq_rotate_quantize(const void* X, const void* R_inter, const void* R_intra,
                                 int64_t M, int64_t d, void* out_codes, void* out_scales,
                                 void* stream);

/* Algorithm 3 steps 1-4 with the rotation in the paper's own structure (Section 5; App. A.7 counts
 * B^2 + K^2 parameters and O(B^2 K) + O(B K^2) work per token): ONE inter-block matrix R_B that
 * mixes the B = d/32 blocks of a token, the same for each of the 32 positions, and ONE intra-block
 * matrix shared by all blocks.  Per token, with X the token's [B, 32] reshape:
 *   Y = R_B X        y[32 b' + k] = sum_b  R_B[b'][b] x[32 b + k]
 *   Z = Y R_intra    z[32 b' + j] = sum_k  y[32 b' + k] R_intra[k][j]
 * then Eq. 1 as in torq_rotate_quantize (same output layouts).  Equivalent to torq_rotate_quantize
 * with R_inter = kron(R_B^T, I_32) and R_intra repeated for every block, at 2 d (B + 32) instead of
 * 2 d^2 flop per token.
 *   X [M, d] bf16;  R_B [d/32, d/32] bf16 (required);  R_intra [32, 32] bf16 or NULL = identity
 * Requires d % 256 == 0, 16-byte aligned pointers.  fp32 accumulation: step 2 on the tensor cores
 * with exact bf16 products, step 3 on the tensor cores as well, with y split exactly into three
 * bf16 terms against the bf16 R_intra.  R_B is a constant of the layer like R_inter (see the
 * conventions above). */
torq_status torq_rotate_quantize_structured(const void* X, const void* R_B, const void* R_intra,
                                            int64_t M, int64_t d, void* out_codes, void* out_scales,
                                            void* stream);

/* Algorithm 3 steps 1-5 with the structured rotation: torq_rotate_quantize_structured into
 * `workspace` (codes [M, d/2], then 256-byte aligned the tiled scales; >= M*d/2 rounded up to 256
 * plus torq_scales_bytes(M, d) bytes, 256-byte aligned), then torq_mxfp4_gemm against weights that
 * were rotated with the same R_B and R_intra offline.  dbg_codes / dbg_scales as in
 * torq_rotated_linear.  Requires d % 256 == 0 and N % 8 == 0. */
torq_status torq_rotated_linear_structured(const void* X, const void* R_B, const void* R_intra,
                                           const void* Wq, const void* Ws, int64_t M, int64_t d,
                                           int64_t N, void* Y, torq_dtype y_dtype, void* workspace,
                                           size_t workspace_bytes, void* dbg_codes, void* dbg_scales,
                                           void* stream);

/* Algorithm 3 step 5 (option B): Y[m,n] = sum_k a^[m,k] w^[n,k], a^/w^ the dequantized MXFP4
 * values (codeword x 2^e), fp32 accumulation on the block-scaled FP4 tensor cores.
 *   Aq [M, K/2] u8, As scales of A (tiled, torq_scales_bytes(M, K))
 *   Wq [N, K/2] u8 (the fused weight W' stored with K contiguous), Ws (tiled, (N, K))
 *   Y  [M, N] row-major of y_dtype
 * Requires M,N >= 1, K % 128 == 0, N % 8 == 0, 16-byte aligned pointers. */
torq_status torq_mxfp4_gemm(const void* Aq, const void* As, const void* Wq, const void* Ws,
                            int64_t M, int64_t N, int64_t K, void* Y, torq_dtype y_dtype,
                            void* stream);

/* Algorithm 3 steps 1-5 in one call: rotate, quantize, multiply.  The quantized activations live
 * in `workspace` (>= torq_workspace_bytes(M, d, N) bytes, 256-byte aligned), laid out as codes
 * [M, d/2] followed (256-byte aligned) by the tiled scales; pass dbg_codes / dbg_scales non-NULL
 * to also receive copies of them.  Up to 256 tokens the rotation is one kernel that splits its
 * contraction over thread-block clusters and adds the partial sums on chip, in a fixed order.
 * Beyond that, when the rotation has few output tiles (128 rows x 256 columns each) relative to
 * the number of SMs -- a narrow layer -- the workspace also holds fp32 partial tiles: the rotation
 * is then split along its contraction so that every SM streams a share of R_inter, and a second
 * kernel adds the partials in a fixed order before the intra-block step and Eq. 1.
 * Requires d % 128 == 0 and N % 8 == 0. */
torq_status torq_rotated_linear(const void* X, const void* R_inter, const void* R_intra,
                                const void* Wq, const void* Ws, int64_t M, int64_t d, int64_t N,
                                void* Y, torq_dtype y_dtype, void* workspace,
                                size_t workspace_bytes, void* dbg_codes, void* dbg_scales,
                                void* stream);

/* The whole layer for callers that must not allocate device memory.  (No counterpart in the
 * paper: this exists for the library's users, not for the method.)
 *
 * torq_rotated_linear needs a scratch buffer for the quantized activations, and normally the
 * caller allocates it.  Some callers cannot: a plug-in or custom operator that an inference
 * engine hands nothing but input and output pointers; a serving process whose whole device
 * budget was given to a KV-cache pool at start-up, where a late cudaMalloc fails or evicts;
 * a latency-critical decode loop, where the implicit device-wide synchronisation of
 * cudaMalloc / cudaFree is not acceptable.  For them this entry point keeps the scratch in a
 * fixed array of TORQ_STATIC_WORKSPACE_BYTES that is part of the library image: every device
 * that loads the library holds those bytes from load until the process exits, used or not.
 * The call itself allocates nothing and frees nothing, on the host or the device, and neither
 * does anything it calls.
 *
 * Same arguments, layouts and results as torq_rotated_linear without its workspace and debug
 * parameters.  A problem whose quantized activations (M * d / 2 code bytes rounded up to 256,
 * plus torq_scales_bytes(M, d)) exceed TORQ_STATIC_WORKSPACE_BYTES is refused with
 * TORQ_ERR_WORKSPACE before anything is launched (for example M = 2048, d = 14336 fits;
 * M = 8192, d = 5120 does not).  What is left of the array serves as the split-K scratch of the
 * few-token path when it is large enough.
 *
 * First call on each device: the library looks up the array's device address (and, if no other
 * entry point ran before, performs the one-time per-device set-up every entry point shares).
 * Make that first call during start-up, outside any stream capture.
 *
 * All calls on a device share the one array, and it keeps whatever the previous call left.
 * Nothing in it has to start at zero: the rotation step rewrites every code and scale byte the
 * multiplication step reads before it reads them, so stale contents are never observed.  But two
 * calls that can overlap on the GPU (different streams, or different host threads without
 * ordering between them) write the same bytes and race; run them in one stream or order them
 * with events.  Calls on different devices do not interact. */
#define TORQ_STATIC_WORKSPACE_BYTES (16u << 20)
torq_status torq_rotated_linear_static(const void* X, const void* R_inter, const void* R_intra,
                                       const void* Wq, const void* Ws, int64_t M, int64_t d,
                                       int64_t N, void* Y, torq_dtype y_dtype, void* stream);

/* Eq. 1 alone: quantize Z [M, d] (fp32 or bf16) to MXFP4.  On fp32 input the result is defined
 * bit for bit (round to nearest even on the e2m1 grid, saturation to +-6, sign bit kept). */
torq_status torq_quantize_mxfp4(const void* Z, torq_dtype z_dtype, int64_t M, int64_t d,
                                void* out_codes, void* out_scales, void* stream);

/* Scale-factor layout (not in the paper; fixed by the FP4 tensor-core instruction): 512-byte tiles
 * of 128 rows x 4 K-blocks, tiles ordered row-tile major; inside a tile
 *   byte = (row % 32) * 16 + ((row % 128) / 32) * 4 + (kblock % 4).
 * Host-side pure functions. */
size_t torq_scales_bytes(int64_t rows, int64_t k);
size_t torq_scale_offset(int64_t row, int64_t kblock, int64_t k);
size_t torq_workspace_bytes(int64_t M, int64_t d, int64_t N);

/* Re-tile a plain [rows, k/32] scale matrix into the layout above (padding bytes := 0x00). */
torq_status torq_swizzle_scales(const void* linear_scales, int64_t rows, int64_t k, void* out,
                                void* stream);

/* Offline helper for the weight side of step 5 (W' = R~^T W, R~ = R_inter . blockdiag(R_intra)):
 * writes R~ [d, d] as fp32 computed in fp32 from the bf16 inputs.  d % 32 == 0. */
torq_status torq_merge_rotations(const void* R_inter, const void* R_intra, int64_t d,
                                 void* R_merged_f32, void* stream);

/* The same merged matrix rounded once (nearest even) to bfloat16: the operand of the one-GEMM form
 * of the rotation, torq_rotate_quantize(X, R_merged, NULL), which Section 5 writes as
 * R = R_inter (x) R_intra.  That form is a different quantized operator from the two-level one (the
 * rounding of R~ to bfloat16 moves about one code in a thousand). */
torq_status torq_merge_rotations_bf16(const void* R_inter, const void* R_intra, int64_t d,
                                      void* R_merged_bf16, void* stream);

/* Algorithm 3 step 5, option B ("weight fusion"), the offline weight side: W' = R~^T W with
 * R~ = R_inter . blockdiag(R_intra), stored as [N, d] (K = d contiguous), then quantized along K
 * (Section 6.1: weights and activations are both quantized).
 *   W        [d, N] float32 row-major (out = x W)
 *   R_inter  [d, d] bf16 (required), R_intra [d/32, 32, 32] bf16 or NULL = identity
 *   Wq [N, d/2] u8, Ws torq_scales_bytes(N, d) bytes: the operands torq_mxfp4_gemm takes
 *   workspace: torq_prepare_weights_workspace_bytes(d, N) bytes (10 N d, rounded up), 256-byte aligned
 * Row n of W' is (W^T[n, :] R_inter) R_intra per block, i.e. steps 2-3 applied to the rows of W^T:
 * W^T is split exactly into three bfloat16 terms and the rotation kernels contract all of them against
 * R_inter in one fp32 accumulation on the tensor cores (every product exact); the intra-block step
 * is fp32 FMAs; the result is quantized by the kernel behind torq_quantize_mxfp4.  d % 64 == 0.
 * Three launches (split, rotation, quantizer).  Not on the inference path. */
size_t torq_prepare_weights_workspace_bytes(int64_t d, int64_t N);
torq_status torq_prepare_weights(const void* W, const void* R_inter, const void* R_intra, int64_t d,
                                 int64_t N, void* Wq, void* Ws, void* workspace, size_t workspace_bytes,
                                 void* stream);

/* ---- NVFP4 variant (the paper's format study, Section 6 "Generalizability to Other Formats") -----
 * The same layer with NVFP4 operands: e2m1 codes as above, blocks of 16 along K, one FP8 E4M3
 * scale byte per (row, block) and one float32 scale per tensor; x^ = codeword * e4m3(byte) *
 * tensor_scale.  The paper names the format and reports accuracies only; the arithmetic below is
 * the library's definition (each step one IEEE float32 operation, round to nearest even):
 *   c = 1 / (6 tensor_scale);  byte = E4M3(amax_block * c), saturating at 448;
 *   r = 1 / (e4m3(byte) * tensor_scale), or 0 when byte == 0;  code = e2m1(z * r), saturating at
 *   6, sign of z kept.
 * The tensor scale is an input (calibrated beforehand; amax(tensor) / (6 * 448) uses the whole
 * E4M3 range) and must be positive and finite.  Scale bytes use the tiled layout of
 * torq_scale_offset with 16-element blocks: a buffer has torq_nvfp4_scales_bytes(rows, k) bytes,
 * the byte of (row, block c) sits at torq_scale_offset(row, c, 2 * k); padding bytes are 0x00
 * (E4M3 zero).  The intra-block rotation acts inside a quantization block, so it is [d/16, 16, 16]
 * here; the rotation kernels take it in 32-wide block-diagonal form, made once by
 * torq_expand_intra16. */
size_t torq_nvfp4_scales_bytes(int64_t rows, int64_t k);
size_t torq_nvfp4_workspace_bytes(int64_t M, int64_t d, int64_t N);

/* R_intra16 [d/16, 16, 16] bf16 -> R_intra32 [d/32, 32, 32] bf16: blocks 2b and 2b+1 on the diagonal of
 * block b, zeros elsewhere.  d % 32 == 0. */
torq_status torq_expand_intra16(const void* R_intra16, int64_t d, void* R_intra32, void* stream);

/* torq_prepare_weights in NVFP4 (R_intra32 as for torq_rotate_quantize_nvfp4).  The tensor scale is
 * max |W'| / (6 * 448) (one float32 division), found by a reduction on the device and written to
 * *tensor_scale (HOST pointer): this call therefore synchronises `stream` once, between the
 * rotation and the quantization.  An all-zero W' has no scale: TORQ_ERR_SHAPE.
 * Ws: torq_nvfp4_scales_bytes(N, d) bytes. */
torq_status torq_prepare_weights_nvfp4(const void* W, const void* R_inter, const void* R_intra32, int64_t d,
                                       int64_t N, void* Wq, void* Ws, float* tensor_scale, void* workspace,
                                       size_t workspace_bytes, void* stream);

/* Quantize Z [M, d] (fp32 or bf16) to NVFP4; d % 16 == 0.  Bit-exact by the definition above. */
torq_status torq_quantize_nvfp4(const void* Z, torq_dtype z_dtype, int64_t M, int64_t d,
                                float tensor_scale, void* out_codes, void* out_scales, void* stream);

/* Algorithm 3 steps 1-4 with the NVFP4 quantizer.  X [M, d] bf16; R_inter [d, d] bf16 (required);
 * R_intra32 [d/32, 32, 32] bf16 or NULL = identity; d % 32 == 0.  Outputs as torq_quantize_nvfp4. */
torq_status torq_rotate_quantize_nvfp4(const void* X, const void* R_inter, const void* R_intra32,
                                       int64_t M, int64_t d, float tensor_scale, void* out_codes,
                                       void* out_scales, void* stream);

/* torq_rotate_quantize_structured with the NVFP4 quantizer at its end: the rotation in the paper's own
 * structure (R_B across blocks, one shared R_intra [32, 32] -- for a 16-wide intra rotation its two
 * 16 x 16 blocks on the diagonal -- or NULL) and 16-element blocks with E4M3 scales.  d % 256 == 0. */
torq_status torq_rotate_quantize_structured_nvfp4(const void* X, const void* R_B, const void* R_intra,
                                                  int64_t M, int64_t d, float tensor_scale,
                                                  void* out_codes, void* out_scales, void* stream);

/* Algorithm 3 step 5 on NVFP4 operands: Y[m,n] = a_tensor_scale * w_tensor_scale *
 * sum_k (code * e4m3 scale)_a[m,k] (code * e4m3 scale)_w[n,k], fp32 accumulation on the tensor
 * cores (kind::mxf4nvf4, 16-element blocks).  Shapes and layouts as torq_mxfp4_gemm with
 * 16-element blocks: K % 128 == 0, N % 8 == 0. */
torq_status torq_nvfp4_gemm(const void* Aq, const void* As, float a_tensor_scale, const void* Wq,
                            const void* Ws, float w_tensor_scale, int64_t M, int64_t N, int64_t K,
                            void* Y, torq_dtype y_dtype, void* stream);

/* Steps 1-5 in NVFP4: torq_rotate_quantize_nvfp4 into `workspace` (at least
 * torq_nvfp4_workspace_bytes(M, d, N) bytes, 256-byte aligned), then torq_nvfp4_gemm.  As in
 * torq_rotated_linear, for few tokens the workspace also holds the fp32 partial tiles of the
 * rotation split along its contraction.  d % 128 == 0, N % 8 == 0. */
torq_status torq_rotated_linear_nvfp4(const void* X, const void* R_inter, const void* R_intra32,
                                      float x_tensor_scale, const void* Wq, const void* Ws,
                                      float w_tensor_scale, int64_t M, int64_t d, int64_t N, void* Y,
                                      torq_dtype y_dtype, void* workspace, size_t workspace_bytes,
                                      void* dbg_codes, void* dbg_scales, void* stream);

/* ---- MXINT4 variant (the paper's format study, Section 6 "Generalizability to Other Formats") ----
 * The same layer with integer elements: blocks of 32 along K, one E8M0 scale byte per block by
 * the same rule and in the same tiled layout as MXFP4 (torq_scales_bytes / torq_scale_offset),
 * elements q = clamp(rint(z / 2^e), -7, 7) (rint = round half to even; z / 2^e is exact, so the
 * quantizer is bit-exact by definition); decoding x^ = q * 2^e.
 * Two forms of the codes:
 *   stored form   [rows, k/2] bytes: two's-complement nibbles, even element in the low nibble;
 *   operand form  [rows, k]   bytes: the FP8 E4M3 byte whose value is q (a zero may carry a sign
 *                 bit).  The tensor cores of this GPU have no 4-bit integer path; the GEMM runs
 *                 as tcgen05.mma kind::mxf8f6f4 on E4M3 operands with the E8M0 block scales.
 *                 Integer products and their power-of-two scales are exact in it; accumulation
 *                 is fp32.
 * The rotation entry points write the operand form directly.  All pointers device, 16-byte
 * aligned; errors as elsewhere in this header.  The paper has no worked example of this format. */
size_t torq_mxint4_workspace_bytes(int64_t M, int64_t d, int64_t N);

/* torq_prepare_weights in MXINT4: Wn [N, d/2] stored form and / or W8 [N, d] operand form (either
 * may be NULL, not both), Ws torq_scales_bytes(N, d) bytes. */
torq_status torq_prepare_weights_mxint4(const void* W, const void* R_inter, const void* R_intra, int64_t d,
                                        int64_t N, void* Wn, void* W8, void* Ws, void* workspace,
                                        size_t workspace_bytes, void* stream);

/* Quantize Z [M, d] (fp32 or bf16), d % 32 == 0.  packed != 0: stored form, out_codes [M, d/2];
 * packed == 0: operand form, out_codes [M, d].  out_scales: torq_scales_bytes(M, d) bytes. */
torq_status torq_quantize_mxint4(const void* Z, torq_dtype z_dtype, int64_t M, int64_t d, int packed,
                                 void* out_codes, void* out_scales, void* stream);

/* Stored form [rows, k/2] -> operand form [rows, k] (nibble -8 becomes the E4M3 byte of -8). */
torq_status torq_mxint4_expand(const void* packed, int64_t rows, int64_t k, void* out_bytes, void* stream);

/* Algorithm 3 steps 1-4 with the MXINT4 quantizer.  X [M, d] bf16; R_inter [d, d] bf16 (required);
 * R_intra [d/32, 32, 32] bf16 or NULL = identity; d % 32 == 0.  out_bytes [M, d] operand form. */
torq_status torq_rotate_quantize_mxint4(const void* X, const void* R_inter, const void* R_intra, int64_t M,
                                        int64_t d, void* out_bytes, void* out_scales, void* stream);

/* torq_rotate_quantize_structured with the MXINT4 quantizer at its end (R_B [d/32, d/32] bf16, one
 * shared R_intra [32, 32] bf16 or NULL; d % 256 == 0).  out_bytes [M, d] operand form. */
torq_status torq_rotate_quantize_structured_mxint4(const void* X, const void* R_B, const void* R_intra,
                                                   int64_t M, int64_t d, void* out_bytes, void* out_scales,
                                                   void* stream);

/* Algorithm 3 step 5 on MXINT4 operands: Y[m,n] = sum_k a^[m,k] w^[n,k].  A8 [M, K], W8 [N, K]
 * operand form; As, Ws tiled E8M0 scales; K % 128 == 0, N % 8 == 0; Y [M, N] fp32 or bf16. */
torq_status torq_mxint4_gemm(const void* A8, const void* As, const void* W8, const void* Ws, int64_t M,
                             int64_t N, int64_t K, void* Y, torq_dtype y_dtype, void* stream);

/* Steps 1-5 in MXINT4: torq_rotate_quantize_mxint4 into `workspace` (at least
 * torq_mxint4_workspace_bytes(M, d, N) bytes, 256-byte aligned), then torq_mxint4_gemm.  As in
 * torq_rotated_linear, few tokens take the rotation split along its contraction, its fp32 partial
 * sums in the same workspace.  dbg_bytes
 * [M, d] / dbg_scales, when not NULL, receive copies of the quantized activations.
 * d % 128 == 0, N % 8 == 0. */
torq_status torq_rotated_linear_mxint4(const void* X, const void* R_inter, const void* R_intra, const void* W8,
                                       const void* Ws, int64_t M, int64_t d, int64_t N, void* Y,
                                       torq_dtype y_dtype, void* workspace, size_t workspace_bytes,
                                       void* dbg_bytes, void* dbg_scales, void* stream);

/* ---- calibration of the inter-block rotation (Section 5.1; offline, not on the inference path) ----
 * Covariance across the blocks of a token, pooled over the T calibration tokens and the 32
 * positions of a block (block means taken as zero, as Section 5.1 assumes):
 *   Sigma[b, b'] = (1 / (32 T)) sum_t sum_k x[t, 32 b + k] x[t, 32 b' + k]
 * X [T, d] bf16, Sigma_f64 [d/32, d/32] float64 (written whole); d % 32 == 0.  float64 accumulation. */
torq_status torq_block_covariance(const void* X, int64_t T, int64_t d, void* Sigma_f64, void* stream);

/* Algorithm 1 (Givens rotations for variance equalisation): an orthogonal Q with
 * diag(Q Sigma Q^T) = (tr Sigma / B) 1 up to the absolute threshold eps -- the matrix R_B that
 * torq_rotate_quantize_structured applies across the blocks of a token.  Departures from the
 * listing, which cannot reach its own stated output as printed: the rotation angle is the one that
 * sets sigma_ii to the target exactly (the printed angle zeroes sigma_ij instead and spreads the two
 * variances); the pair is (largest deviation, smallest deviation), ties to the lowest index; the
 * matrix returned is the transpose of the listing's accumulated product, so that the output line
 * holds as written.  At most B - 1 rotations.
 *   Sigma_f64 [B, B] float64: in Sigma, out Q Sigma Q^T;  Q_f64 [B, B] float64;
 *   Q_bf16 [B, B] bf16 or NULL (Q rounded through float32);  n_rotations: device int32 or NULL.
 * One CTA; float64, one rounding per operation (no fused multiply-add), so the result is defined
 * bit for bit.  1 <= B <= 32768, eps >= 0. */
torq_status torq_givens_equalize(void* Sigma_f64, int64_t B, double eps, void* Q_f64, void* Q_bf16,
                                 void* n_rotations, void* stream);

/* Measurement tool (no counterpart in the paper): runs `groups` groups of four block-scaled FP4
 * tensor-core instructions (256 x 256 x 64 each, the GEMM's own instruction) per CTA pair on operands
 * that already sit in shared memory, with no loads and no epilogue, times them with CUDA events on
 * `stream`, synchronises, and writes the rate in TFLOP/s to *tflops (host pointer).  This is the
 * issue-bound peak of the FP4 tensor pipe on the device at hand: the denominator for the GEMM's
 * roofline fraction where no vendor-measured FP4 peak exists.  Includes the kernel's launch, so use
 * groups >= 20000 (about a millisecond). */
torq_status torq_probe_fp4_peak(int groups, double* tflops, void* stream);

/* Self-test of the bounded device waits (no counterpart in the paper).  Every wait inside the
 * tensor-core kernels gives up after 2 s, latches TORQ_ERR_TIMEOUT, lets the kernel's other warps
 * drain and returns; a healthy run never takes that path.  This call runs it on purpose in a
 * one-CTA kernel whose two barriers nothing ever arrives on: one warp's wait runs out after
 * `limit_ns` (1 us .. 100 ms) and latches the error word with wait-site id 7, the other warp's wait
 * (2 s limit) must leave through the CTA's abort flag.  Nothing faults or hangs: the waits give up
 * by design, and the context stays usable.
 *   result_u64x3: three device uint64: [0] = 1 if the first wait gave up by itself, [1] = 1 if the
 *   second left through the abort flag, [2] = nanoseconds the second one waited.
 * Afterwards torq_last_device_error() returns TORQ_ERR_TIMEOUT | 7 << 8 (and clears the word). */
torq_status torq_selftest_wait_timeout(uint64_t limit_ns, void* result_u64x3, void* stream);

const char* torq_status_string(torq_status s);

/* Synchronises `stream`, then returns and clears the device error word of the current device:
 * 0, or TORQ_ERR_TIMEOUT in the low byte with the id of the wait that gave up in bits 8..15. */
int torq_last_device_error(void* stream);

/* Host helper (no device work): the list of output tiles that the CTA-pair kernels (more than 128
 * rows) walk for a [rows x cols] output on `pairs` CTA pairs (74 on a 148-SM part), in the order
 * in which they are dealt round robin: tile i goes to pair i % pairs.  Tiles are 256 rows high and
 * 256 columns wide; where that leaves the last wave partly empty and cols is a multiple of 256,
 * some row tiles are covered by fewer 256-column tiles followed by 192-column ones (three wide
 * tiles traded for four narrow ones), chosen so that the longest pair finishes earliest.  Both
 * torq_rotate_quantize (cols = d) and torq_mxfp4_gemm (cols = N), and their format variants, use
 * this list.
 *   out: host array of 3 * cap int32, or NULL; receives (row_tile, first_column, width) per tile.
 * Returns the number of tiles (also when it exceeds cap; only cap triples are written), or -1 for
 * rows < 1, cols < 1 or pairs < 1. */
int64_t torq_pair_tile_list(int64_t rows, int64_t cols, int32_t pairs, int32_t* out, int64_t cap);

/* Number of kernels this library has launched since load (all devices, all streams). */
int64_t torq_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* TORQ_H_ */
