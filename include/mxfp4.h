/*
 * mxfp4.h -- C ABI of the B200 (sm_100a) MXFP4 quantize + block-scaled GEMM library.
 *
 * The library implements the hot path of MXFP4 training of transformer linear layers:
 * both GEMM operands are quantized to OCP MXFP4 (E2M1 elements, one E8M0 power-of-two
 * scale per 32 contiguous elements along the reduction axis; Appendix A.1, Eq. (1)),
 * optionally after a 32-point Hadamard rotation along that axis (Appendix A.2), and
 * multiplied on the FP4 tensor cores (Fprop / Dgrad / Wgrad, Appendix C).
 *
 * Conventions for every entry point unless stated otherwise
 *   - All data pointers are DEVICE pointers owned by the caller.  The library allocates
 *     no device memory and keeps no reference to a buffer after the call's work is done.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls only
 *     enqueue work; they do not synchronise.
 *   - Return value: MXFP4_OK (0) or a negative MXFP4_ERR_* code.  Argument errors are
 *     detected on the host before anything is enqueued.  Device-side problems (a bounded
 *     wait that expired) never trap: the kernel records a status word and returns, and
 *     mxfp4_check() reports it.
 *   - A GEMM operand is "K-major": operand[o][k], k contiguous.  Codes hold two elements
 *     per byte, element k even in bits 3:0 and k odd in bits 7:4.  A code is
 *     (sign << 3) | magnitude with magnitudes 0..7 = {0, 0.5, 1, 1.5, 2, 3, 4, 6}.
 *   - A scale byte b means 2^(b - 127).
 *   - Launches use programmatic dependent launch: a kernel's set-up may overlap the tail of the
 *     previous kernel in the stream, and every kernel waits for that kernel's completion before
 *     it touches global memory, so stream order is what a caller observes.  MXFP4_PDL=0 in the
 *     environment (read once) selects plain launches.
 *   - Host threads: per-device state (function attributes, the resident-grid size, the copy
 *     streams and events of the host-buffer layer call, the static scratch address) is created
 *     on first use, once per device, and that set-up is safe against several host threads
 *     making their first call at the same time.  The host-buffer layer calls of one device
 *     share one set of copy streams and events: do not run two of them at the same time.
 */
#ifndef MXFP4_H_
#define MXFP4_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* status codes */
#define MXFP4_OK 0
#define MXFP4_ERR_NULL (-1)      /* a required pointer is NULL                               */
#define MXFP4_ERR_SHAPE (-2)     /* non-positive size (empty tensors are refused, not skipped), K not a
                                    multiple of 32, ld too small, or a size past the kernels' 32-bit tile
                                    arithmetic: a dimension of 2^31 or more, more than 2^30 tiles (128 x 128
                                    source tiles of a quantizer, 256 x 384 output tiles of a GEMM), or 2^31
                                    or more (output tile, 128-element K-step) pairs of a GEMM             */
#define MXFP4_ERR_ALIGN (-3)     /* pointer not 16-byte aligned, or ld not a multiple of 8    */
#define MXFP4_ERR_ENUM (-4)      /* axis / hadamard_mode / rounding / layout / dtype invalid  */
#define MXFP4_ERR_WORKSPACE (-5) /* workspace missing or too small                            */
#define MXFP4_ERR_CUDA (-6)      /* a CUDA runtime/driver call failed (launch, descriptor)    */
#define MXFP4_ERR_TIMEOUT (-7)   /* a bounded device-side wait expired (reported by check)    */
#define MXFP4_ERR_DEVICE (-8)    /* not an sm_100 device                                      */
#define MXFP4_ERR_STATIC_LIMIT (-9) /* mxfp4_linear_static: problem exceeds the built-in scratch */
#define MXFP4_ERR_BOUNDS (-10)   /* bounds-checking debug build only: a kernel computed an address outside
                                    its buffer (reported by check; the access was skipped)              */

/* enums (plain ints in the ABI) */
#define MXFP4_AXIS_ROWS 0 /* 32-blocks run down the rows (column-wise 32x1); operand = src^T */
#define MXFP4_AXIS_COLS 1 /* 32-blocks run along the contiguous axis (row-wise 1x32)         */

#define MXFP4_HADAMARD_NONE 0
#define MXFP4_HADAMARD_DET 1  /* deterministic 32-point rotation                              */
#define MXFP4_HADAMARD_RAND 2 /* sign diagonal from `seed`, then the rotation                 */
#define MXFP4_HADAMARD_DET16 3  /* two 16-point rotations per 32-block (the paper's H16)      */
#define MXFP4_HADAMARD_RAND16 4 /* 16 signs from `seed` (same for both halves), then H16      */

#define MXFP4_ROUND_RNE 0 /* round to nearest, ties to even                                   */
#define MXFP4_ROUND_SR 1  /* stochastic rounding, Philox4x32-10 keyed by (seed, element)      */

#define MXFP4_SCALES_CANONICAL 0 /* scales[o][t], row-major, outer x K/32 bytes               */
#define MXFP4_SCALES_TILED 1     /* 128-row x 4-block tiles of 512 bytes (what the GEMM reads)*/

#define MXFP4_BLOCK_1X32 0  /* one scale per 32 elements along K (Appendix D, 1D)               */
#define MXFP4_BLOCK_32X32 1 /* one scale per 32 operand rows x 32 elements (Appendix D, 2D)      */

#define MXFP4_PRECISION_MXFP4 0 /* E2M1 elements, the method's GEMMs                              */
#define MXFP4_PRECISION_MXFP8 1 /* E4M3 elements, the passes the ladder of Table 1 leaves in FP8  */
#define MXFP4_PRECISION_MXFP4_32X32 2 /* MXFP4 with Appendix D's 32 x 32 blocks for both operands */

#define MXFP4_OUT_BF16 0
#define MXFP4_OUT_FP32 1

#define MXFP4_PASS_FPROP 0
#define MXFP4_PASS_DGRAD 1
#define MXFP4_PASS_WGRAD 2

/* Library version (major * 100 + minor). */
int mxfp4_version(void);

/* Human-readable name of a status code (static storage). */
const char* mxfp4_status_string(int status);

/* Bytes of packed codes for an operand of `outer` rows and K elements per row: outer*K/2. */
size_t mxfp4_codes_bytes(int64_t outer, int64_t K);

/*
 * Bytes of the scale buffer.  Canonical: outer*K/32.  Tiled: whole tiles of 128 rows x 4
 * blocks, ceil(outer/128) * ceil(K/128) * 512 bytes; the scale of (row o, block t) lives at
 *   ((o/128) * ceil(K/128) + t/4) * 512 + (o%32)*16 + ((o%128)/32)*4 + (t%4).
 * Padding rows / blocks hold 0 (the scale of an all-zero block).  Returns 0 on bad input.
 */
size_t mxfp4_scales_bytes(int64_t outer, int64_t K, int scale_layout);

/*
 * mxfp4_quantize -- Eq. (1) of Appendix A.1 with the optional rotation of Appendix A.2,
 * for row-wise (axis 1) or column-wise (axis 0) 32-blocks (Appendix D).
 *
 *   src_bf16     [rows x cols] bf16, row-major, leading dimension ld_src (elements,
 *                multiple of 8, >= cols); 16-byte aligned.
 *   axis         MXFP4_AXIS_COLS: operand[o][k] = src[o][k], outer = rows, K = cols.
 *                MXFP4_AXIS_ROWS: operand[o][k] = src[k][o], outer = cols, K = rows -- the
 *                transposed operand Dgrad (W^T) and Wgrad (dY^T, X^T) need, written directly
 *                with no separate transpose pass.
 *   K must be a multiple of 32; outer may be any positive number (cols need not be a multiple
 *                of 8 for MXFP4_AXIS_ROWS: only ld_src has that rule).
 *   hadamard_mode, rounding, seed: each 32-block v becomes H*v (mode 1) or H*(D*v) (mode 2,
 *                D the +-1 diagonal drawn from `seed`) in fp32 with a fixed five-stage
 *                butterfly; modes 3 / 4 rotate each half of the block with its own 16-point
 *                transform instead (the same butterfly without its last stage); the block scale is 2^(floor(log2 amax) - 2); elements are rounded
 *                to E2M1 with saturation at 6.  With MXFP4_ROUND_SR each element uses 8 bits
 *                of Philox4x32-10(key = (lo32(seed), hi32(seed)), counter = (lo32(g), hi32(g),
 *                operand_tag, 0)) with g = e >> 4 and e the element's 64-bit index o*K + k in
 *                the operand view: byte (e & 3) of output word ((e & 15) >> 2).
 *   operand_tag  decorrelates the stochastic-rounding streams of different operands.
 *   codes        out, [outer x K/2] bytes, 16-byte aligned.
 *   scales       out, mxfp4_scales_bytes(outer, K, scale_layout) bytes, 16-byte aligned.
 * Inputs must be finite; with a rotation the 32-term (16-term) sums of a block must stay finite
 * in fp32 too, i.e. magnitudes below about 1e37 (overflowing blocks are outside the contract: the
 * result is then unspecified, never a fault).
 */
int mxfp4_quantize(const void* src_bf16, int64_t rows, int64_t cols, int64_t ld_src, int axis,
                   int hadamard_mode, int rounding, uint64_t seed, uint32_t operand_tag,
                   void* codes, void* scales, int scale_layout, void* stream);

/*
 * mxfp4_quantize_2d -- mxfp4_quantize with the 32 x 32 block strategy of Appendix D: one E8M0
 * scale is shared by 32 consecutive operand rows x one 32-element block along K (regions aligned
 * to multiples of 32 both ways; a last region may have fewer rows).  The scale comes from the
 * largest magnitude in the region -- of the rotated values when hadamard_mode != 0 -- and is
 * written into the scale entry of every row of the region, so codes and scales have exactly the
 * format of mxfp4_quantize and feed mxfp4_gemm unchanged.  With hadamard_mode 0 the result is
 * transpose-invariant: axis ROWS gives the transposed codes and scales of axis COLS.
 * Arguments, shapes, alignment and errors as mxfp4_quantize.
 */
int mxfp4_quantize_2d(const void* src_bf16, int64_t rows, int64_t cols, int64_t ld_src, int axis,
                      int hadamard_mode, int rounding, uint64_t seed, uint32_t operand_tag,
                      void* codes, void* scales, int scale_layout, void* stream);

/*
 * mxfp4_quantize_dual -- both orientations of one tensor from ONE read of it (Appendix D; a
 * linear layer uses each of X, W, dY once blocked along its rows and once down its columns,
 * Appendix C).  Writes
 *   codes_rowwise / scales_rowwise : the operand of mxfp4_quantize(axis = MXFP4_AXIS_COLS),
 *                                    [rows x cols/2] bytes, stochastic-rounding tag tag_rowwise;
 *   codes_colwise / scales_colwise : the operand of mxfp4_quantize(axis = MXFP4_AXIS_ROWS),
 *                                    the transposed operand [cols x rows/2] bytes, tag tag_colwise;
 * each bit-identical to the single-axis call (block_shape MXFP4_BLOCK_1X32) or to
 * mxfp4_quantize_2d (MXFP4_BLOCK_32X32) with the same rotation, rounding and seed.
 * rows and cols must both be multiples of 32 (both are reduction axes), ld_src a multiple of 8;
 * all five pointers are device pointers, 16-byte aligned; scale buffers are sized with
 * mxfp4_scales_bytes(rows, cols, layout) and mxfp4_scales_bytes(cols, rows, layout).
 * Algorithmic traffic: 2 + 2 * (1/2 + 1/32) = 3.0625 bytes per element instead of 5.0625 for
 * two single-axis calls.  Nothing is launched on error.
 */
int mxfp4_quantize_dual(const void* src_bf16, int64_t rows, int64_t cols, int64_t ld_src, int hadamard_mode,
                        int rounding, uint64_t seed, uint32_t tag_rowwise, uint32_t tag_colwise,
                        int block_shape, void* codes_rowwise, void* scales_rowwise, void* codes_colwise,
                        void* scales_colwise, int scale_layout, void* stream);

/*
 * mxfp4_quantize_pair -- mxfp4_quantize for two tensors in ONE kernel launch (the two operands
 * of a linear pass, Appendix D: both are quantized along the GEMM's reduction axis).  The result
 * for each tensor is bit-identical to its own mxfp4_quantize call; rotation, rounding and seed are
 * shared, the operand tags are per tensor.  `a` and `b` point to HOST structs; every pointer
 * inside them is a DEVICE pointer with the alignment and shape rules of mxfp4_quantize.
 * Supported axis pairs (a, b): (COLS, COLS), (COLS, ROWS), (ROWS, ROWS) -- the three a linear
 * layer's passes need; any other returns MXFP4_ERR_ENUM.  Nothing is launched on error.
 */
typedef struct mxfp4_quant_desc {
    const void* src_bf16;   /* device, [rows x cols] bf16 row-major                 */
    int64_t rows, cols, ld_src;
    int32_t axis;           /* MXFP4_AXIS_COLS / MXFP4_AXIS_ROWS                     */
    uint32_t operand_tag;
    void* codes;            /* device out, [outer x K/2] bytes                      */
    void* scales;           /* device out, mxfp4_scales_bytes(outer, K, layout)     */
} mxfp4_quant_desc;

int mxfp4_quantize_pair(const mxfp4_quant_desc* a, const mxfp4_quant_desc* b, int hadamard_mode,
                        int rounding, uint64_t seed, int scale_layout, void* stream);

/*
 * mxfp4_gemm -- the block-scaled product the linear layers run in place of their FP8 GEMM
 * (Appendix A.2 last paragraph; operand orientation per Appendix C):
 *   out[m][n] = alpha * sum_t 2^(sa[m][t]-127) * 2^(sb[n][t]-127) * sum_{k in block t} A[m][k]*B[n][k]
 * A: [M x K], B: [N x K], both K-major codes with TILED scales (as mxfp4_quantize writes
 * them).  K multiple of 32.  Products are exact; accumulation is fp32 on the tensor cores, which
 * truncate: a sum of K/64 steps is low in magnitude by at most (K/64) * 2^-23 times its largest
 * partial sum -- about 1e-6 * sum|products| at K = 28672 on products of mixed sign, 1e-5 on
 * products that all have one sign.
 * Scale bytes of tile rows past M (or N) are never used for a stored element and may hold
 * anything; the bytes of blocks past K/32 inside the last 128-element tile are multiplied with
 * zero codes and must not be 0xFF (mxfp4_quantize writes 0 there).
 *   alpha        exact power of two in the intended use (2^-5 undoes H*H^T = 32*I).
 *   out          [M x N] row-major, leading dimension ld_out (elements), bf16 (RNE) or fp32;
 *                16-byte aligned, ld_out*sizeof(elem) a multiple of 16.
 *   workspace    unused by the current kernel; may be NULL with workspace_bytes 0.
 */
int mxfp4_gemm(const void* a_codes, const void* a_scales, const void* b_codes,
               const void* b_scales, int64_t M, int64_t N, int64_t K, float alpha, void* out,
               int out_dtype, int64_t ld_out, void* workspace, size_t workspace_bytes,
               void* stream);

/*
 * Workspace (device bytes) the fused linear passes need for the two quantized operands:
 * codes + tiled scales of both, each region 256-byte aligned.  pass = MXFP4_PASS_*.
 */
size_t mxfp4_linear_workspace_bytes(int64_t T, int64_t in_features, int64_t out_features, int pass);

/*
 * Fused linear passes (Appendix C).  Each quantizes its two operands along the reduction
 * axis (same hadamard_mode / rounding / seed for both so that the rotation cancels;
 * operand_tag 0 for the first operand, 1 for the second) and runs the GEMM with
 * alpha = 2^-5 when rotated with H32, 2^-4 with H16, 1 otherwise.  All matrices row-major and dense (ld = width).
 *   fprop: Y[T x out]   = X[T x in]    * W[out x in]^T   (both row-wise along `in`)
 *   dgrad: dX[T x in]   = dY[T x out]  * W[out x in]     (dY row-wise along `out`; W column-wise)
 *   wgrad: dW[out x in] = dY[T x out]^T * X[T x in]      (both column-wise along tokens)
 * The reduction size (in / out / T respectively) must be a multiple of 32, all widths
 * multiples of 8.  workspace >= mxfp4_linear_workspace_bytes(...), 256-byte aligned.
 */
int mxfp4_linear_fprop(const void* X, const void* W, void* Y, int64_t T, int64_t in_features,
                       int64_t out_features, int hadamard_mode, int rounding, uint64_t seed,
                       int out_dtype, void* workspace, size_t workspace_bytes, void* stream);
int mxfp4_linear_dgrad(const void* dY, const void* W, void* dX, int64_t T, int64_t in_features,
                       int64_t out_features, int hadamard_mode, int rounding, uint64_t seed,
                       int out_dtype, void* workspace, size_t workspace_bytes, void* stream);
int mxfp4_linear_wgrad(const void* dY, const void* X, void* dW, int64_t T, int64_t in_features,
                       int64_t out_features, int hadamard_mode, int rounding, uint64_t seed,
                       int out_dtype, void* workspace, size_t workspace_bytes, void* stream);

/*
 * The 8-bit side of the precision ladder (Table 1: Fprop, Dgrad and Wgrad are switched to MXFP4
 * one by one; the others stay in FP8).  The paper does not say which FP8 recipe its baseline
 * uses; this library's 8-bit passes are MXFP8 -- Eq. (1) of Appendix A.1 with E4M3 elements:
 * one E8M0 scale 2^(floor(log2 amax) - 8) per 32 elements along the reduction axis, elements
 * rounded to the nearest E4M3 value (ties to even, saturating at 448, sign kept on zero), no
 * rotation and no stochastic rounding.
 *
 * mxfp4_quantize_fp8: as mxfp4_quantize; codes are [outer x K] bytes (one E4M3 code per element),
 *   scales as for the 4-bit format (same size, same layouts).
 * mxfp4_gemm_fp8: as mxfp4_gemm on such operands (tcgen05 kind::mxf8f6f4, fp32 accumulation).
 * mxfp4_linear_pass: one pass at a chosen precision; (a, b, out) = (X, W, Y) / (dY, W, dX) /
 *   (dY, X, dW) for MXFP4_PASS_FPROP / _DGRAD / _WGRAD.  With MXFP4_PRECISION_MXFP4 it is
 *   mxfp4_linear_fprop / _dgrad / _wgrad; MXFP4_PRECISION_MXFP4_32X32 is the same pass with both
 *   operands quantized by mxfp4_quantize_2d; with MXFP4_PRECISION_MXFP8 hadamard_mode, rounding and
 *   seed are ignored.  Workspace: mxfp4_linear_pass_workspace_bytes (0 for a bad argument).
 * Errors as for the 4-bit entry points.
 */
int mxfp4_quantize_fp8(const void* src_bf16, int64_t rows, int64_t cols, int64_t ld_src, int axis, void* codes,
                       void* scales, int scale_layout, void* stream);
int mxfp4_gemm_fp8(const void* a_codes, const void* a_scales, const void* b_codes, const void* b_scales,
                   int64_t M, int64_t N, int64_t K, float alpha, void* out, int out_dtype, int64_t ld_out,
                   void* stream);
size_t mxfp4_linear_pass_workspace_bytes(int64_t T, int64_t in_features, int64_t out_features, int pass,
                                         int precision);
int mxfp4_linear_pass(int pass, int precision, const void* a, const void* b, void* out, int64_t T,
                      int64_t in_features, int64_t out_features, int hadamard_mode, int rounding, uint64_t seed,
                      int out_dtype, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Layer-level form of the same three passes (Appendix C), each tensor read ONCE: a linear layer
 * uses X, W and dY each in both block orientations (X: Fprop + Wgrad, W: Fprop + Dgrad,
 * dY: Dgrad + Wgrad), so the forward call quantizes X and W with mxfp4_quantize_dual, runs the
 * Fprop GEMM and keeps the column-wise operands (X^T, W^T as MXFP4 codes + scales: 0.53 bytes
 * per element instead of the bf16 tensors) in `saved` for the backward call, which quantizes dY
 * once for both of its GEMMs.  Y, dX and dW are bit-identical to mxfp4_linear_fprop / _dgrad /
 * _wgrad with the same rotation, rounding and seed (same operand tags, same kernels).
 *   T, in_features, out_features  all multiples of 32.
 *   saved      device, mxfp4_linear_layer_bytes(.., MXFP4_LAYER_SAVED) bytes, 256-byte aligned;
 *              written by forward, read by backward (the caller keeps it alive in between).
 *   workspace  device scratch, mxfp4_linear_layer_bytes(.., MXFP4_LAYER_FORWARD / _BACKWARD)
 *              bytes, 256-byte aligned; free again once the call's work has run on `stream`.
 *   dx_dtype, dw_dtype  MXFP4_OUT_*.
 * Launches: forward 2 quantize + 1 GEMM, backward 1 quantize + 2 GEMMs (5 for the layer's three
 * passes instead of 6, and 3.06 instead of 5.06 bytes of quantize traffic per element).
 * mxfp4_linear_layer_bytes returns 0 for a bad argument.
 */
#define MXFP4_LAYER_SAVED 0
#define MXFP4_LAYER_FORWARD 1
#define MXFP4_LAYER_BACKWARD 2
size_t mxfp4_linear_layer_bytes(int64_t T, int64_t in_features, int64_t out_features, int which);
int mxfp4_linear_forward(const void* X, const void* W, void* Y, int64_t T, int64_t in_features,
                         int64_t out_features, int hadamard_mode, int rounding, uint64_t seed, int out_dtype,
                         void* saved, size_t saved_bytes, void* workspace, size_t workspace_bytes, void* stream);
int mxfp4_linear_backward(const void* dY, void* dX, void* dW, int64_t T, int64_t in_features,
                          int64_t out_features, int hadamard_mode, int rounding, uint64_t seed, int dx_dtype,
                          int dw_dtype, const void* saved, size_t saved_bytes, void* workspace,
                          size_t workspace_bytes, void* stream);

/*
 * Host-buffer form of the three passes: a_host / b_host / out_host are HOST pointers (pinned
 * memory makes the copies asynchronous).  The call copies both inputs to the caller's device
 * staging buffers, runs the pass there, copies the result back and returns after the
 * stream has drained, so out_host is valid on return.
 *   pass        MXFP4_PASS_*; (a, b, out) = (X, W, Y) / (dY, W, dX) / (dY, X, dW).
 *   dev_a, dev_b, dev_out   device staging for the two inputs (bf16) and the output.
 */
int mxfp4_linear_host(int pass, const void* a_host, const void* b_host, void* out_host, int64_t T,
                      int64_t in_features, int64_t out_features, int hadamard_mode, int rounding,
                      uint64_t seed, int out_dtype, void* dev_a, void* dev_b, void* dev_out,
                      void* workspace, size_t workspace_bytes, void* stream);

/*
 * Host-buffer form of mxfp4_linear_forward + mxfp4_linear_backward for one linear layer: the six
 * *_host pointers are HOST buffers (pinned memory makes the copies asynchronous and lets them
 * overlap), every other pointer is a DEVICE buffer the caller owns.  X, W and dY cross the bus
 * once each (the per-pass form copies every tensor twice), on a copy stream of the library's
 * own in the order they are needed; the kernels run on `stream`; Y, dX and dW return on a second
 * copy stream, each as soon as its GEMM has finished, so results flow out while dY still flows
 * in.  With drain != 0 the call returns after everything has drained: the three host outputs are
 * valid.  With drain == 0 it returns as soon as the work is queued, so that the next layer's
 * inputs travel while this layer's kernels run and its results are still on their way back.
 * Consecutive calls order themselves buffer by buffer, assuming that they pass the same staging
 * buffers in the same roles and the same `stream`: an input staging buffer is overwritten once the
 * previous call's quantize launch has read it, an output staging buffer once the previous call's
 * copy to the host has left it.  No other work may use the staging buffers while such calls are
 * in flight.  The host outputs of all undrained calls are valid after
 * mxfp4_linear_layer_host_drain(stream), and the host inputs must stay untouched until then.
 *   dev_x, dev_w, dev_dy    device staging for the bf16 inputs ([T x in], [out x in], [T x out]);
 *   dev_y, dev_dx, dev_dw   device staging for the outputs; all six distinct;
 *   saved, workspace        as for forward / backward; workspace must cover the larger of
 *                           MXFP4_LAYER_FORWARD and MXFP4_LAYER_BACKWARD.
 * The library creates its two copy streams and its events on first use per device and keeps them.
 * Outputs are bit-identical to the device-buffer calls.
 */
int mxfp4_linear_layer_host(const void* X_host, const void* W_host, const void* dY_host, void* Y_host,
                            void* dX_host, void* dW_host, int64_t T, int64_t in_features, int64_t out_features,
                            int hadamard_mode, int rounding, uint64_t seed, int y_dtype, int dx_dtype, int dw_dtype,
                            void* dev_x, void* dev_w, void* dev_dy, void* dev_y, void* dev_dx, void* dev_dw,
                            void* saved, size_t saved_bytes, void* workspace, size_t workspace_bytes, void* stream,
                            int drain);
int mxfp4_linear_layer_host_drain(void* stream);

/*
 * mxfp4_linear_static -- the fused passes for callers that cannot allocate device memory.
 * (The paper has no counterpart to this entry point; it exists for integration only.)
 *
 * Who needs it: code that runs where neither cudaMalloc nor the host framework's allocator may
 * be called -- for example a callback inside a runtime that has handed all device memory to
 * its own arena (cudaMalloc would fail or fragment it), a latency-critical serving loop that
 * cannot afford cudaMalloc's implicit device synchronisation, or a plugin that is given
 * input/output buffers but no allocator handle.  Such callers still pass the inputs and the
 * output; only the scratch for the two quantized operands comes from the library.
 *
 * How: the scratch is a fixed array of MXFP4_STATIC_SCRATCH_BYTES that is part of the library
 * image, so every GPU that loads the library holds that much memory until the process exits.
 * The call allocates nothing (no cudaMalloc / cudaFree, no allocating library routine).
 *
 *   pass, (a, b, out), T, in_features, out_features, hadamard_mode, rounding, seed, out_dtype:
 *       exactly as mxfp4_linear_fprop / _dgrad / _wgrad (pass = MXFP4_PASS_*), same results.
 *   Limit: mxfp4_linear_workspace_bytes(T, in, out, pass) must not exceed
 *       MXFP4_STATIC_SCRATCH_BYTES; larger problems return MXFP4_ERR_STATIC_LIMIT and nothing
 *       is enqueued (use the workspace-taking entry points for those).
 *   First call on a device: looks up the array's device address (once per device, with that
 *       device current).  Make that first call before any stream capture begins.
 *   Sharing: every call on a device uses the same array and finds the previous call's
 *       contents in it.  Nothing needs clearing -- each call rewrites all bytes it later reads --
 *       but two calls that overlap on the GPU (different streams, or concurrent host threads
 *       without ordering) race on the array.  Issue them on one stream or order them with events.
 */
#define MXFP4_STATIC_SCRATCH_BYTES (16 * 1024 * 1024)
int mxfp4_linear_static(int pass, const void* a, const void* b, void* out, int64_t T,
                        int64_t in_features, int64_t out_features, int hadamard_mode, int rounding,
                        uint64_t seed, int out_dtype, void* stream);

/*
 * Synchronises `stream` and returns the sticky device-side status of the current device:
 * MXFP4_OK, MXFP4_ERR_TIMEOUT (a kernel gave up a bounded wait; its output is invalid) or
 * MXFP4_ERR_CUDA.  The status word is cleared by the call.
 */
int mxfp4_check(void* stream);

/*
 * Self-test of the error path (no counterpart in the paper): enqueues a one-warp kernel whose
 * only wait can never be satisfied and is limited to a few hundred attempts.  The kernel gives
 * up within microseconds, records the time-out and returns normally -- nothing traps, faults
 * or hangs -- so the next mxfp4_check(stream) returns MXFP4_ERR_TIMEOUT (and clears it).
 */
int mxfp4_selftest_wait_timeout(void* stream);

/*
 * The library can be built with -DMXFP4_BOUNDS (no counterpart in the paper): a debug build that
 * stands in for a memory sanitizer.  Every shared-memory access whose address a kernel computes is
 * then checked against the buffer it belongs to (range and natural alignment); a miss is skipped
 * and recorded, and the next mxfp4_check returns MXFP4_ERR_BOUNDS.  Results are bit-identical to
 * the normal build.  mxfp4_bounds_checked() tells which build is loaded (1 / 0);
 * mxfp4_selftest_bounds enqueues a one-thread kernel that hands the checker an address one
 * element past a buffer -- the address is only tested, never dereferenced, in either build -- so
 * that the next mxfp4_check(stream) returns MXFP4_ERR_BOUNDS (and clears it).
 */
int mxfp4_bounds_checked(void);
int mxfp4_selftest_bounds(void* stream);

/*
 * Diagnostic (no counterpart in the paper): enqueues one launch of a kernel that issues the GEMM's
 * own pair MMAs (256 x 192 x 64, kind::mxf4.block_scale, eight per iteration = one K-step) on
 * operands resident in shared memory -- no loads, no epilogue -- on every CTA pair of the device.
 * Timed by the caller (CUDA events around a few launches) it gives the ceiling the tensor pipe
 * sets for MXFP4 on this device: with constant operand bits the clock-bound rate, with
 * random_operands != 0 the rate the power limit allows once operands toggle.  *flops (host, may
 * be NULL) receives the floating-point operations of the launch.  iterations: 1..20000 (a launch
 * of 10000 takes about 5 ms).  Every wait inside is bounded.
 */
int mxfp4_probe_mma_rate(int iterations, int random_operands, void* stream, double* flops);

#ifdef __cplusplus
}
#endif
#endif /* MXFP4_H_ */
