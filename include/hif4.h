/*
 * hif4.h -- C ABI of the HiF4 (HiFloat4) W4A4 linear-layer hot path for NVIDIA B200 (sm_100a).
 *
 * HiF4 is the 4-bit block floating-point format of "HiFloat4 Format for Language Model
 * Inference" (Section II).  One HiF4 *unit* stores 64 values in 288 bits: 32 bits of shared
 * three-level scaling metadata plus 64 four-bit sign-magnitude S1P2 elements (Section II-A,
 * Table I, Table II: 4.5 bits per value).
 *
 * ---------------------------------------------------------------------------------------------
 * Unit layout in memory (36 bytes, 4-byte aligned, units of a row consecutive, rows consecutive).
 * The paper's figure of the unit is not reproduced in its text, so this byte order is a
 * convention of this library:
 *
 *   bytes 0..3   little-endian uint32 `meta`
 *                  bits  7:0   E6M2 level-1 scale byte `eeeeee mm` (Table I): value
 *                              2^(e-48) * (1 + m/4); 0xFF is NaN, there is no zero or infinity
 *                  bits 15:8   E1_8  level-2 micro-exponents, bit 8+j  covers elements 8j..8j+7
 *                  bits 31:16  E1_16 level-3 micro-exponents, bit 16+k covers elements 4k..4k+3
 *   bytes 4..35  S1P2 codes, element i in byte 4 + i/2, low nibble for even i, high nibble for
 *                odd i; nibble = sign<<3 | magnitude, magnitude m in 0..7 meaning m/4.
 *
 * Value of element i (Eq. 2, 0-based indices):
 *   V_i = (-1)^sign * (m/4) * 2^(E1_8[i/8] + E1_16[i/4]) * E6M2,   all 64 are NaN if E6M2 is NaN.
 * ---------------------------------------------------------------------------------------------
 *
 * Conventions common to every call
 *   - All data pointers are DEVICE pointers unless a parameter says "host".  The caller owns every
 *     buffer; the library never allocates, frees or synchronises (hif4_last_device_status is the
 *     one documented exception and synchronises the stream it is given).
 *   - Every call is asynchronous on `stream` (a cudaStream_t passed as void* so that this header
 *     needs no CUDA header; NULL is the legacy default stream).
 *   - The return value is a status code.  Argument errors are found on the host before any launch.
 *     NaN and Inf in the data are not errors; they encode as the format defines.
 *   - Matrices are row-major.  Both GEMM operands are quantised along K (units contiguous in K),
 *     because Eq. 3 pairs unit k of a row of A with unit k of a row of B.  A weight W[K_in, N_out]
 *     is therefore handed over as its transpose [N, K].
 */
#ifndef HIF4_H_
#define HIF4_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define HIF4_UNIT_ELEMS 64   /* elements per unit (Section II-A)                    */
#define HIF4_UNIT_BYTES 36   /* 4 metadata bytes + 32 code bytes = 288 bits         */

typedef enum {
  HIF4_OK = 0,
  HIF4_ERR_NULL = 1,           /* a required pointer is NULL                                   */
  HIF4_ERR_SHAPE = 2,          /* negative size, cols or K not a multiple of 64, ld too small  */
  HIF4_ERR_ALIGN = 3,          /* pointer or leading dimension breaks the stated alignment     */
  HIF4_ERR_DTYPE = 4,          /* unknown hif4_dtype / hif4_round value                        */
  HIF4_ERR_WORKSPACE = 5,      /* workspace smaller than hif4_*_workspace reports              */
  HIF4_ERR_CUDA = 6,           /* a CUDA call or launch failed; cudaGetLastError keeps the code*/
  HIF4_ERR_DEVICE_TIMEOUT = 7, /* a bounded wait inside a kernel ran out (see last_device_status) */
  HIF4_ERR_UNSUPPORTED = 8     /* valid request that this build does not implement             */
} hif4_status;

/* HIF4_FP16 is a source type only (hif4_quantize, hif4_linear): Section II-B extends the conversion to
 * further source types and names FP32 and FP16; FP16 arithmetic cannot hold the reciprocal of an
 * E6M2 scale (up to 2^48), so FP16 elements are widened exactly to FP32 and Algorithm 1 runs in FP32
 * arithmetic.  hif4_dequantize returns HIF4_ERR_DTYPE for it (HiF4's range exceeds FP16's).  */
typedef enum { HIF4_BF16 = 0, HIF4_FP32 = 1, HIF4_FP16 = 2 } hif4_dtype;

/* Rounding used where Algorithm 1 rounds to E6M2 and to S1P2 (Section II-B allows half-to-even or
 * half-away-from-zero).  Products inside the algorithm always round to
 * nearest-even.  */
typedef enum { HIF4_RNE = 0, HIF4_RHA = 1 } hif4_round;

/* Bytes of the packed form of a [rows, cols] matrix: rows * (cols/64) * 36 (Section II-A).
 * Returns 0 when cols is not a multiple of 64 or a size is negative.  Host-only, no GPU use.  */
size_t hif4_packed_bytes(int64_t rows, int64_t cols);

/* hif4_quantize -- Algorithm 1 (Section II-B) applied to every 64-element unit of a matrix.
 *   src        device, [rows, cols] of `dt`, row stride `ld_src` ELEMENTS (>= cols); base and row
 *              stride must keep every row 16-byte aligned.
 *   dst_units  device, rows*(cols/64) units of 36 bytes, row-major, 4-byte aligned (16-byte aligned
 *              storage gives the fastest stores).  Fully overwritten.
 *   mode       HIF4_RNE or HIF4_RHA.
 * The working precision of the algorithm is that of the source type (BF16 arithmetic for BF16
 * input, FP32 arithmetic for FP32 and FP16 input).  A unit holding a NaN becomes the canonical NaN unit
 * (meta 0x000000FF, codes 0).  rows == 0 or cols == 0 is a no-op returning HIF4_OK.  */
hif4_status hif4_quantize(const void* src, hif4_dtype dt, int64_t rows, int64_t cols,
                          int64_t ld_src, void* dst_units, hif4_round mode, void* stream);

/* hif4_quantize_transposed -- the same conversion with the units running down the columns: unit r of
 * column c holds src[64 r .. 64 r + 63][c], i.e. dst is hif4_quantize of the transposed matrix without the
 * transpose ever being written.  (Algorithm 1 converts 64 values at a time and does not say how those
 * 64 lie in memory; Eq. 3 needs both GEMM operands cut along the contraction dimension, so a matrix
 * that is contracted along its rows -- a weight kept as [K, N], or any operand of a transposed product --
 * is quantized this way.)
 *   src        device, [rows, cols] of `dt` (any source type of hif4_quantize, same working precision), row
 *              stride `ld_src` elements (>= cols), rows 16-byte aligned; rows must be a multiple of 64, cols
 *              a multiple of 8.
 *   dst_units  device, cols*(rows/64) units, column-major in the sense above ([cols, rows/64, 36 bytes]),
 *              4-byte aligned.  Fully overwritten.  */
hif4_status hif4_quantize_transposed(const void* src, hif4_dtype dt, int64_t rows, int64_t cols,
                                     int64_t ld_src, void* dst_units, hif4_round mode, void* stream);

/* hif4_dequantize -- Eq. 2 for every element; exact in BF16 and FP32.
 *   src_units  device, rows*(cols/64) units, 4-byte aligned.
 *   dst        device, [rows, cols] of `dt`, row stride `ld_dst` elements (>= cols), rows 16-byte
 *              aligned.  Fully overwritten inside [rows, cols]; padding beyond cols is untouched.  */
hif4_status hif4_dequantize(const void* src_units, int64_t rows, int64_t cols, void* dst,
                            hif4_dtype dt, int64_t ld_dst, void* stream);

/* Workspace (device scratch) that hif4_gemm needs for this shape on the current device; may be 0.
 * For M <= 32 it holds the decoded activation rows (2 * K * 8, 16 or 32 bytes); for larger M a few KB of
 * completion words when tiles are split along K.  The figure is the largest need over all kernels that
 * could serve the shape, so it stays valid whatever path is chosen at call time.  Host-only.  */
hif4_status hif4_gemm_workspace(int64_t M, int64_t N, int64_t K, size_t* bytes);

/* hif4_gemm -- C = A * B^T with A, B in HiF4 and FP32 accumulation: C[i][j] is the sum over the
 * K/64 unit pairs of Eq. 3's dot product of unit k of row i of A with unit k of row j of B.
 *   A_units    device, [M, K/64] units.        B_units  device, [N, K/64] units.
 *   C          device, [M, N] FP32, row stride `ldc` elements (>= N), 4-byte aligned; 16-byte
 *              aligned rows (base % 16 == 0 and ldc % 4 == 0) allow vector stores.  Overwritten
 *              inside [M, N] (no alpha/beta); padding beyond N is untouched.
 *   workspace  device scratch of at least hif4_gemm_workspace bytes, 256-byte aligned, contents
 *              undefined on entry and exit; may be NULL when 0 bytes are needed.  Calls that may run
 *              at the same time (different streams) need workspaces of their own.
 * K must be a multiple of 64.  M == 0 or N == 0 is a no-op; K == 0 zero-fills C.
 * Units whose E6M2 byte is NaN make every C entry they touch NaN.  */
hif4_status hif4_gemm(const void* A_units, const void* B_units, float* C, int64_t M, int64_t N,
                      int64_t K, int64_t ldc, void* workspace, size_t workspace_bytes,
                      void* stream);

/* hif4_linear -- the W4A4 linear layer in one call (Section IV: every linear layer's activations
 * are converted to HiF4 before the matrix multiplication): Y = HiF4(X) * W^T, i.e. hif4_quantize of the
 * activations (Algorithm 1) followed by hif4_gemm with pre-quantized weights (Eq. 3), in stream order.
 *   X          device, [M, K] of `dt` (BF16 or FP32), row stride ld_x elements, rows 16-byte aligned.
 *   W_units    device, [N, K/64] units (the weight quantized along K beforehand).
 *   Y          device, [M, N] FP32, row stride ldy.
 *   workspace  device scratch of at least hif4_linear_workspace bytes, 256-byte aligned: holds the
 *              packed activations (and what hif4_gemm needs for this shape).
 * The result is bit-identical to calling hif4_quantize and hif4_gemm one after the other.  */
hif4_status hif4_linear_workspace(int64_t M, int64_t N, int64_t K, size_t* bytes);
hif4_status hif4_linear(const void* X, hif4_dtype dt, int64_t ld_x, const void* W_units, float* Y, int64_t M,
                        int64_t N, int64_t K, int64_t ldy, hif4_round mode, void* workspace,
                        size_t workspace_bytes, void* stream);

hif4_status hif4_grouped_gemm_workspace(int num_groups, int64_t total_rows, int64_t N, int64_t K,
                                        size_t* bytes);

/* hif4_grouped_gemm -- the same contraction per group g (an MoE expert, Section IV-B converts the
 * MoE linears):  C[off[g]:off[g+1], :] = A[off[g]:off[g+1], :] * B[g]^T.
 *   A_units            device, [total_rows, K/64] units, rows sorted by group.
 *   B_units            device, [num_groups, N, K/64] units.
 *   C                  device, [total_rows, N] FP32, row stride ldc.
 *   group_offsets_dev  device, num_groups+1 int64 prefix sums, off[0] = 0, off[num_groups] =
 *                      total_rows, non-decreasing.  Read by the kernel only: routing results never
 *                      return to the host.  Empty groups are allowed.  */
hif4_status hif4_grouped_gemm(const void* A_units, const void* B_units, float* C,
                              const int64_t* group_offsets_dev, int num_groups, int64_t total_rows,
                              int64_t N, int64_t K, int64_t ldc, void* workspace,
                              size_t workspace_bytes, void* stream);

/* hif4_grouped_gemm_noalloc -- hif4_grouped_gemm without a workspace argument.  (The paper has no
 * counterpart: this is a packaging variant of the call above, not another operation.)
 *
 * For callers that cannot allocate device memory: code running under a fixed memory plan that was
 * sized at start-up, a plug-in that receives tensors but no allocator, or a section where the
 * device-wide synchronisation of a cudaMalloc is not acceptable.  The tile table that the
 * tensor-core kernel needs lives in a __device__ array of HIF4_NOALLOC_SCRATCH_BYTES bytes inside
 * the library; every GPU that loads the library holds it until the process exits.  The call itself
 * performs no cudaMalloc / cudaFree and uses no allocating library routine.
 *
 *   Arguments are those of hif4_grouped_gemm.  The result meets the same tolerance; it comes from the
 *   single-CTA tensor-core kernel (128-row tiles), whereas hif4_grouped_gemm normally runs the CTA-pair
 *   kernel, so the FP32 summation order and therefore the last bits of C may differ between the two.
 *   Limit     ceil(total_rows / 128) + num_groups table entries of 16 bytes, rounded up to 256,
 *             must fit in HIF4_NOALLOC_SCRATCH_BYTES (65536: e.g. 256 groups and 491520 rows);
 *             beyond that the call returns HIF4_ERR_WORKSPACE and launches nothing.
 *   Sharing   all calls on one GPU use the same array.  Calls ordered on one stream are safe (each
 *             call rewrites every entry it reads; nothing has to be zero beforehand).  Calls that
 *             may overlap on the GPU -- different streams or host threads without ordering -- race
 *             on the table and produce wrong results.
 *   Set-up    the first call on each GPU looks up the array's device address
 *             (cudaGetSymbolAddress, with that GPU current) and keeps it; make that first call
 *             outside any stream capture.
 * hif4_debug_set_gemm_path does not apply to this call.  */
#define HIF4_NOALLOC_SCRATCH_BYTES 65536
hif4_status hif4_grouped_gemm_noalloc(const void* A_units, const void* B_units, float* C,
                                      const int64_t* group_offsets_dev, int num_groups,
                                      int64_t total_rows, int64_t N, int64_t K, int64_t ldc,
                                      void* stream);

/* Size in bytes of the built-in scratch array (HIF4_NOALLOC_SCRATCH_BYTES).  Host-only.  */
size_t hif4_grouped_gemm_noalloc_capacity(void);

/* hif4_mse_roundtrip -- the quantization-error experiment of Section III-A for one tensor: convert a BF16 tensor
 * to a 4-bit block format and back, write the image as FP32 and sum the squared error against the source.
 *   HIF4_FMT_HIF4       Algorithm 1 (round-half-to-even), then Eq. 2
 *   HIF4_FMT_MXFP4      blocks of 32, power-of-two scale 2^(floor(log2 amax) - 2), E2M1 elements
 *   HIF4_FMT_NVFP4      blocks of 16, E4M3 scale = amax / 6, E2M1 elements ("direct cast")
 *   HIF4_FMT_NVFP4_PTS  NVFP4 after per-tensor scaling of the peak magnitude to 2688, undone afterwards
 * (E2M1 and E4M3 rounding to nearest, ties to even, saturating; every step one FP32 operation.)
 *   src_bf16    device, n BF16 elements, 16-byte aligned; n a multiple of 64.
 *   dst         device, n FP32 elements receiving the image, or NULL when only the error is wanted.
 *   sq_err_sum  device, one FP64: sum over the elements of (image - source)^2, accumulated in FP64 in an order
 *               that does not depend on scheduling.
 *   workspace   device scratch of at least hif4_mse_workspace bytes, 256-byte aligned.  */
typedef enum { HIF4_FMT_HIF4 = 0, HIF4_FMT_MXFP4 = 1, HIF4_FMT_NVFP4 = 2, HIF4_FMT_NVFP4_PTS = 3 } hif4_bfp4_format;
hif4_status hif4_mse_workspace(int64_t n, hif4_bfp4_format fmt, size_t* bytes);
hif4_status hif4_mse_roundtrip(const void* src_bf16, int64_t n, hif4_bfp4_format fmt, float* dst, double* sq_err_sum,
                               void* workspace, size_t workspace_bytes, void* stream);

/* Synchronises `stream` and returns HIF4_ERR_DEVICE_TIMEOUT if any kernel of this library gave up
 * a bounded wait since the last call (the flag is cleared), HIF4_ERR_CUDA if the stream reports
 * an error, else HIF4_OK.  For tests and debugging.  */
hif4_status hif4_last_device_status(void* stream);

/* Static, NUL-terminated description of a status code.  Host-only.  */
const char* hif4_status_string(hif4_status s);

/* ---------------------------------------------------------------------------------------------
 * Test and benchmark hooks (hif4_debug_*).  Not part of the product surface: nothing above depends on
 * them except that hif4_gemm honours the path override while it is set.
 *
 * hif4_debug_set_gemm_path: 0 = choose the GEMM kernel by shape (default), 1 = CUDA-core kernel only,
 * 2 = the single-CTA tensor-core (tcgen05) kernel whenever it is legal (K % 256 == 0, 16-byte aligned
 * operands), even for small M, 3 = the CTA-pair tensor-core kernel (256 x 256 tiles) whenever it is legal,
 * 4 = the weight-streaming kernel whenever it is legal (M <= 32), 5 = the variant of that kernel that follows
 * Eq. 3's factorisation (FP8 E4M3 tensor-core operands holding the elements with their micro-exponents, the two
 * level-1 scales applied to each unit pair's sum) whenever it is legal (M <= 32), 6 = hif4_linear converts BF16
 * activations inside the CTA-pair kernel whenever that is legal (M > 128).  Process-wide and not thread-safe.
 * hif4_gemm_workspace does not depend on it: it always reports the largest need over all paths.
 *
 * hif4_debug_launch_count: number of kernels this library has launched in this process (monotonic,
 * host-side counter).  */
hif4_status hif4_debug_set_gemm_path(int path);
uint64_t hif4_debug_launch_count(void);

/* hif4_debug_wait_timeout: launches a one-block kernel that waits on an mbarrier nobody arrives on, with the
 * same bounded-wait helper the GEMM kernels use but a budget of `budget_ns` (1 .. 100 000 000) instead of their
 * 2 s.  The wait runs out, the kernel raises the device error word and returns normally; the next
 * hif4_last_device_status on that stream returns HIF4_ERR_DEVICE_TIMEOUT, the one after it HIF4_OK.  Nothing
 * faults or hangs: no copy or MMA is in flight.  (The paper has no counterpart; this exercises the library's
 * failure reporting.)  */
hif4_status hif4_debug_wait_timeout(uint64_t budget_ns, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* HIF4_H_ */
