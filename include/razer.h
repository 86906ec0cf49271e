/*
 * razer.h - C ABI of the B200 (sm_100a) RaZeR matmul library.
 *
 * RaZeR (arXiv 2501.04052) stores a tensor as FP4-E2M1 codes in blocks of 16 along K.
 * Each block has one 8-bit scale byte and the tensor has one FP32 scale (Sec. 3,
 * Eq. 1-3).  FP4 has two zero codes; one of them is remapped, per block, to a special
 * value chosen from a small set of allowed values, and the unused top bit(s) of the
 * scale byte say which one (Sec. 4.1, 4.2, Eq. 6-7).
 *
 * Conventions shared by every entry point
 *   y[m, n] = sum_k x[m, k] * W[n, k]      W is N x K, x is M x K, K contiguous in both.
 *   Interchange format of a quantized tensor (what a quantizer emits, what
 *   razer_pack_layout and razer_decode_act read):
 *     codes  uint8 [rows][K/2]   element k = 2j in bits 3:0, k = 2j+1 in bits 7:4 of byte j;
 *                                nibble = S E1 E0 M (Eq. 5)
 *     scales uint8 [rows][K/16]  weights     : [sv_sign | sv_select | E2 E1 E0 | M2 M1 M0]
 *                                              6-bit scale = an E4M3 code (Eq. 4) with E3 = 0
 *                                activations : [sv_sign | E3 E2 E1 E0 | M2 M1 M0]
 *     special value of a block = (sv_sign ? -1 : +1) * sv_mag[sv_select]   (Sec. 4.4)
 *     element value            = special value if code == remap_code,
 *                                0 if code is the other zero code, else Eq. 5
 *     dequantized element      = tensor_scale * block_scale * element value   (Sec. 3)
 *   All pointers named *_dev are DEVICE pointers; *_host are HOST pointers.  The caller
 *   owns every buffer; no entry point allocates, frees or keeps device memory, and none
 *   synchronizes the stream unless its comment says so.  `stream` is a cudaStream_t
 *   passed as void* (NULL = the default stream).  bf16 tensors are raw 16-bit patterns.
 *   Every function returns RAZER_OK (0) or a negative RAZER_ERR_* code, never throws;
 *   razer_last_error() returns a description of the calling thread's last failure.
 *   Stream ordering: the matmul kernels are launched with programmatic dependent launch
 *   (RAZER_PDL=0 in the environment turns it off).  They read the PACKED WEIGHTS before the
 *   kernel directly ahead of them on the stream is known to have finished, and everything
 *   else (activations, outputs, workspace, scale scalars) after it.  Guaranteed: weights
 *   written by razer_pack_layout, by a copy (cudaMemcpyAsync) or by anything that is not the
 *   immediately preceding kernel of the stream are seen.  Not guaranteed: weights written by
 *   a caller's own kernel launched directly ahead of the matmul; put any other operation
 *   between the two (razer_pack_layout does so itself).
 */
#ifndef RAZER_H_
#define RAZER_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  RAZER_OK = 0,
  RAZER_ERR_INVALID_ARG = -1,   /* null pointer, bad size, misaligned buffer               */
  RAZER_ERR_UNSUPPORTED = -2,   /* a block size / special value / mode this build lacks     */
  RAZER_ERR_WORKSPACE = -3,     /* workspace missing or smaller than razer_workspace_bytes  */
  RAZER_ERR_CUDA = -4,          /* a CUDA runtime/driver call failed (text in last_error)   */
  RAZER_ERR_DEVICE_TIMEOUT = -5 /* a bounded device-side wait gave up (status word set)     */
};

enum { RAZER_SCALE_E3M3_META2 = 0,   /* weights: 6-bit scale + 2 metadata bits (Sec. 4.1)  */
       RAZER_SCALE_E4M3_META1 = 1 }; /* activations: 7-bit scale + 1 metadata bit          */

enum { RAZER_OP_GEMV = 0, RAZER_OP_GEMM = 1, RAZER_OP_GEMM_W4A4 = 2 };

/* Description of one RaZeR-quantized weight tensor (host struct, passed by pointer). */
typedef struct razer_desc {
  int32_t N;            /* rows (output features), >= 1                                     */
  int32_t K;            /* columns (reduction dim), multiple of 16                          */
  int32_t block;        /* elements per scale block along K: 16 (Sec. 3) or 32, 64, 128
                           (the block-size study of Sec. 5); K must be a multiple of it      */
  int32_t scale_fmt;    /* RAZER_SCALE_E3M3_META2 for weights                                */
  int32_t remap_code;   /* which zero nibble is the special value in the interchange codes:
                           0x8 (negative zero, default) or 0x0                               */
  float sv_mag[2];      /* special-value magnitudes selected by sv_select; each must be one
                           of 2.5 3.5 4.5 5 5.5 6.5 7 7.5 8 9 10 12 (App. D.3)              */
  float tensor_scale;   /* the FP32 per-tensor scale of Eq. 1                                */
} razer_desc;

/* Text of the calling thread's most recent error ("" if none). Never NULL. */
const char* razer_last_error(void);

/* Library/ABI version: major*10000 + minor*100 + patch. */
int razer_version(void);

/* Number of CUDA kernels this library has launched in this process so far (all threads).
 * Lets a harness report how many device launches a timed region contained. */
unsigned long long razer_kernel_launches(void);

/* Size in bytes of the GPU-internal packed form of the tensor `d` describes.
 * The packed form has 4.5 bits per weight (codes + one scale byte per 16 elements: the byte
 * of a larger block is repeated, so that every kernel reads one layout), padded to whole
 * 128-row x 64-column tiles. */
int razer_packed_bytes(const razer_desc* d, size_t* bytes_out);

/* Offline weight shuffle (Sec. 4.3: weights are reordered once so that the kernels' loads
 * are contiguous).  Reads the interchange format (codes_dev: N*K/2 bytes, scales_dev:
 * N*K/16 bytes) and writes the packed form (razer_packed_bytes bytes, 16-byte aligned).
 * Inside the packed form the remapped code is always 0x8 and blocks whose special value is
 * positive are stored negated with a flag in the scale byte; both are lossless.
 * Asynchronous on `stream`.
 * The matmul entry points begin to read packed_dev before the single kernel directly ahead of
 * them on the stream is known to have finished (programmatic dependent launch; RAZER_PDL=0 in
 * the environment turns that off).  razer_pack_layout therefore queues an empty kernel behind
 * its own, so its output is always safe to use; a caller that fills packed_dev with a kernel of
 * its own must put some other operation between that kernel and the matmul. */
int razer_pack_layout(const razer_desc* d, const uint8_t* codes_dev, const uint8_t* scales_dev,
                      void* packed_dev, void* stream);

/* Verification hook: dequantize the packed tensor (Sec. 3: tensor scale x block scale x
 * element value).  out_is_fp32 == 0: bf16 [N][K] of block_scale * element (exact);
 * out_is_fp32 == 1: float [N][K] of fl32(tensor_scale * that) (one FP32 rounding). */
int razer_dequant(const razer_desc* d, const void* packed_dev, void* out_dev, int out_is_fp32,
                  void* stream);

/* Scratch the matmul entry points need for `op` (RAZER_OP_*) with M activation rows.
 * The workspace must be 256-byte aligned and must have been prepared once with
 * razer_workspace_init; the matmul calls leave it prepared, so one workspace can serve any
 * number of calls, shapes included, one after another.  Calls that may overlap on the GPU
 * must not share a workspace. */
int razer_workspace_bytes(const razer_desc* d, int M, int op, size_t* bytes_out);

/* Prepare a workspace: clears the status word and the per-tile arrival counters the
 * stripe reduction (Sec. 4.3, App. E: partial results of stripes are combined through
 * global memory) relies on.  Needed once after allocation, and again after a call returned
 * RAZER_ERR_DEVICE_TIMEOUT or the process was interrupted mid-kernel.  Asynchronous. */
int razer_workspace_init(void* workspace_dev, size_t workspace_bytes, void* stream);

/* Synchronizes `stream` and reads the workspace's device status word: RAZER_OK, or
 * RAZER_ERR_DEVICE_TIMEOUT if a kernel gave up a bounded wait (its output is then
 * undefined; razer_last_error names the wait). */
int razer_workspace_status(const void* workspace_dev, void* stream);

/* Decode GEMV / skinny GEMM (Sec. 4.3: weight-only FP4 x 16-bit kernel, low-batch regime):
 * y[M][N] (bf16) = bf16( tensor_scale * sum_k x[m][k] * block_scale * element ), FP32
 * accumulation, one rounding at the end.  x_dev: bf16 [M][K]; 1 <= M <= 64. */
int razer_gemv(const razer_desc* d, const void* packed_dev, const void* x_dev, int M,
               void* y_dev, void* workspace_dev, size_t workspace_bytes, void* stream);

/* Prefill GEMM (Sec. 4.3, high-batch regime): same result definition, any M >= 1. */
int razer_gemm(const razer_desc* d, const void* packed_dev, const void* x_dev, int M,
               void* y_dev, void* workspace_dev, size_t workspace_bytes, void* stream);

/* razer_gemv with HOST activations and HOST output: copies x (M*K bf16) into
 * x_stage_dev, runs razer_gemv, brings y (M*N bf16) back and synchronizes the stream.
 * x_host / y_host should be pinned for the copies to be asynchronous.  When y_host is
 * pinned memory that the device can address (what cudaHostAlloc / cudaHostRegister give
 * under unified addressing), the kernel stores y straight into it and y_stage_dev is not
 * touched; otherwise y goes through y_stage_dev and one more copy. */
int razer_gemv_host(const razer_desc* d, const void* packed_dev, const void* x_host, int M,
                    void* y_host, void* x_stage_dev, void* y_stage_dev, void* workspace_dev,
                    size_t workspace_bytes, void* stream);

/* razer_gemv for callers that cannot allocate device memory (the paper has no counterpart;
 * this is a deployment convenience of this library).  Some hosts of this code may not call
 * cudaMalloc: a plug-in running inside another framework's memory pool, a real-time loop
 * that must not enter the allocator, code running between a stream-capture begin and end.
 * The other matmul entry points make such callers bring a workspace; this one uses a 4 MiB
 * scratch array built into the library image instead (every GPU that loads the library holds
 * those 4 MiB until the process exits), so the caller passes inputs and outputs only.
 *   1 <= M <= 16.  A shape whose scratch need exceeds the array (tens of millions of rows)
 *   is rejected with RAZER_ERR_UNSUPPORTED and a message naming both sizes.
 *   The first call on each device looks up the array's device address (with that device
 *   current); make that first call outside any stream capture.  No call allocates or frees.
 *   All calls on one device share the array and it keeps the previous call's contents; the
 *   entry point clears the part that must start at zero on `stream` before the kernel.  Two
 *   calls that can overlap on the GPU (different streams without an ordering between them)
 *   would race on it: order them, or use razer_gemv with separate workspaces.
 *   A device-side wait that gives up leaves y undefined; it is not reported by this entry
 *   point (there is no workspace to query) - use razer_gemv where that matters.
 * Result and argument meaning are those of razer_gemv. */
int razer_gemv_static(const razer_desc* d, const void* packed_dev, const void* x_dev, int M,
                      void* y_dev, void* stream);

/* Online activation quantization (Sec. 4.2: each block is quantized once per allowed
 * special value, +sv_mag and -sv_mag, and the lower squared error wins; Eq. 1-3, 6-7 with
 * the 7-bit E4M3 block scale).  sv_mag = 0 quantizes to plain NVFP4 (Eq. 1-3 alone: no special
 * value, metadata bit clear).  x_dev: bf16 [M][K], K multiple of 16.
 * tensor_scale_in_dev: device float to use as the Eq. 1 scale, or NULL to compute it from
 * the tensor maximum.  In that case amax_scratch_dev is required: two device uint32 (8-byte
 * aligned) that are ZERO before the first call; every call leaves them zero again, so one
 * scratch serves any number of calls one after another (calls that may overlap on the GPU
 * need a scratch each; after a call that was interrupted mid-kernel clear it again).  The
 * whole call is one kernel launch; with a computed scale its CTAs meet once (cooperative
 * launch), and a scale of NaN in tensor_scale_out_dev reports a scratch that was not zero.
 * Writes act_codes_dev [M][K/2], act_scales_dev [M][K/16] in the interchange format
 * (remapped code 0x8) and the scale used to tensor_scale_out_dev. */
int razer_quant_act(const void* x_dev, int M, int K, float sv_mag,
                    const float* tensor_scale_in_dev, uint32_t* amax_scratch_dev,
                    uint8_t* act_codes_dev, uint8_t* act_scales_dev,
                    float* tensor_scale_out_dev, void* stream);

/* Weight quantizer on the GPU (Sec. 4.2, Eq. 1-3 and 6-7 with the 6-bit E3M3 block scale of
 * Sec. 4.1): every block along K is quantized once per allowed special value, in metadata
 * order +sv_mag[0], +sv_mag[1], -sv_mag[0], -sv_mag[1], and the lowest squared error wins
 * (ties: the smaller metadata value).  `block` = elements per scale block along K (16, 32, 64
 * or 128).  scale_aware = 0: all four share the scale of Eq. 2 (block maximum -> 6), as the
 * equations are printed.  scale_aware != 0: a special value beyond 6 whose sign is that of the
 * block's first largest element also competes with a scale of its own (block maximum -> its
 * magnitude); the errors are then compared in the tensor's units and the standard four come
 * first in a tie.  The output format is the same either way.
 * w_dev: FP32 [N][K], K a multiple of `block`, 16-byte aligned.  tensor_scale_in_dev as in
 * razer_quant_act; amax_scratch_dev: one device uint32 (needed when the scale is computed; the
 * call clears it itself).  Writes the interchange format that razer_pack_layout reads:
 * codes_dev [N][K/2], scales_dev [N][K/block] ([meta(2) | E3M3 code(6)]), special value =
 * remap_code (0x8 or 0x0), and the tensor scale to tensor_scale_out_dev.  Every FP32 step is a
 * single IEEE operation in a fixed order, so the result is reproducible bit for bit.
 * Asynchronous on `stream`. */
int razer_quant_weight(const float* w_dev, int N, int K, int block, int scale_aware,
                       const float sv_mag[2], int remap_code,
                       const float* tensor_scale_in_dev, uint32_t* amax_scratch_dev,
                       uint8_t* codes_dev, uint8_t* scales_dev, float* tensor_scale_out_dev,
                       void* stream);

/* Exact decode of RaZeR activations (interchange format, E4M3 scale, one metadata bit) to
 * bf16 [M][K] holding block_scale * element (the tensor scale is NOT applied). */
int razer_decode_act(const uint8_t* act_codes_dev, const uint8_t* act_scales_dev, int M, int K,
                     float sv_mag, void* out_bf16_dev, void* stream);

/* Weight-activation GEMM (App. D.3 setting):
 * y = bf16( w_scale * a_scale * sum_k decoded_act[m][k] * decoded_w[n][k] ).
 * act_codes_dev [M][K/2], act_scales_dev [M][K/16], act_tensor_scale_dev: one device float, as
 * razer_quant_act writes them.  The workspace (RAZER_OP_GEMM_W4A4, zeroed once by
 * razer_workspace_init, 256-byte aligned) is large enough for either path below, but the two
 * lay it out differently: zero it again before a call that takes the other path.
 * use_native_fp4 = 0: both operands RaZeR; the activations are decoded to bf16 (exact) into the
 * workspace and multiplied by the bf16 tensor-core kernel of razer_gemm.
 * use_native_fp4 != 0: the two-pass realization of App. D.3 on the block-scaled FP4 tensor-core
 * instruction (block 16, E4M3 scale factors): the weights are split on the fly into B_main
 * (special value -> signed FP4 base value) and B_comp (signed FP4 remainder, zero elsewhere),
 * both passes accumulate in FP32 into the same accumulator.  RaZeR applies to the weights only:
 * the activations are read as plain NVFP4 (act_sv_mag is ignored, bit 7 of a scale byte is
 * ignored and code 0x8 is a zero), which is what razer_quant_act writes with sv_mag = 0.  Both
 * special-value magnitudes of the descriptor must be sums of two FP4 values (every allowed
 * magnitude is).  Two kernel launches (activation re-layout, matmul). */
int razer_gemm_w4a4(const razer_desc* d, const void* packed_w_dev, const uint8_t* act_codes_dev,
                    const uint8_t* act_scales_dev, const float* act_tensor_scale_dev, float act_sv_mag,
                    int M, void* y_dev, void* workspace_dev, size_t workspace_bytes,
                    int use_native_fp4, void* stream);

/* The same two-pass matmul with the activation operand produced directly in the layout the tensor core reads,
 * the way App. D.3 generates B_main and B_comp "directly in the packed sub-byte layout" its GEMM consumes: no
 * re-layout kernel between quantizer and matmul.
 * razer_fp4_act_bytes: size of that operand for M x K activations (256-byte aligned buffer, caller-owned).
 * razer_quant_act_fp4: plain NVFP4 quantization (Eq. 1-3, the arithmetic of razer_quant_act with sv_mag = 0; same
 * tensor_scale_in_dev / amax_scratch_dev contract, one launch) writing act_fp4_dev: codes padded to whole
 * 256-column stages and scale bytes in the scale-factor tile order of the block-scaled MMA, padding included, so
 * the buffer needs no clearing.  The layout is internal (it depends on the token tile the matmul picks for M).
 * razer_gemm_w4a4_fp4: razer_gemm_w4a4(use_native_fp4 = 1) on such an operand; bit-identical results.  Workspace:
 * RAZER_OP_GEMM_W4A4 (zeroed once by razer_workspace_init). */
int razer_fp4_act_bytes(int M, int K, size_t* bytes_out);
int razer_quant_act_fp4(const void* x_dev, int M, int K, const float* tensor_scale_in_dev,
                        uint32_t* amax_scratch_dev, void* act_fp4_dev, float* tensor_scale_out_dev,
                        void* stream);
int razer_gemm_w4a4_fp4(const razer_desc* d, const void* packed_w_dev, const void* act_fp4_dev,
                        const float* act_tensor_scale_dev, int M, void* y_dev, void* workspace_dev,
                        size_t workspace_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* RAZER_H_ */
