/* liblba: GEMM and 2-D convolution with a low bit-width floating-point accumulator (LBA)
 * on NVIDIA B200 (sm_100a).  C ABI; no CUDA or C++ types appear in any signature.
 *
 * What every call computes, for each output scalar (paper: "Towards Cheaper Inference in
 * Deep Networks with Lower Bit-Width Accumulators"):
 *
 *     y = sum_i x_i * w_i                                             Eq. 3
 *
 * with the fused multiply-add replaced by
 *
 *     FMAq(x, w, s) = Q_acc( Q_prod(x * w) + s )                       Eq. 4
 *
 * where Q is the floating-point quantiser Q^FLOAT_{M,E,b} of Eq. 2 (saturate at
 * R_OF = 2^(2^E-b-1) * (2 - 2^-M), flush to zero below R_UF = 2^-b, no subnormals, mantissa
 * cut to M bits).  The product and the sum inside Eq. 4 are exact; each is rounded once.
 * Inputs are OCP FP8 E4M3 bytes; arithmetic runs on their decoded values ("code domain");
 * real-valued scales are applied to the finished sum in binary32, outside the FMAq unit
 * (Fig. 1, left: W/A quantisation is software, Q_prod/Q_acc are the simulated hardware).
 *
 * Accumulation order (it changes the result, App. D):
 *   LBA_ORDER_SEQUENTIAL  S_0 = 0, S_{i+1} = FMAq(x_i, w_i, S_i), y = S_K       Eq. 8-9
 *   LBA_ORDER_CHUNKED     two hierarchies (Sec. 3, Fig. 1 right, App. D): each run of `chunk`
 *                         consecutive products is accumulated sequentially from 0; the chunk
 *                         sums are then added in chunk order, from 0, with Q_acc after every
 *                         addition (no Q_prod at that level).  The paper uses chunk = 16.
 *                         The last chunk may be short.
 *
 * All device pointers must belong to the current CUDA device.  The library allocates no
 * memory, keeps no state between calls except the last CUDA error code (and the testing hook
 * lba_set_tile_override), and never
 * synchronises: work is enqueued on `stream` (a cudaStream_t passed as void*, NULL = default
 * stream).  Format structs are read on the host during the call.  Because a call only enqueues
 * kernels (and, in the host-buffer variants, asynchronous copies), it may be recorded by a stream
 * capture and replayed from a CUDA graph; the recorded launch shape is the one chosen for the
 * sizes and formats given at capture time.
 *
 * Preconditions that are not checked on the device: no input byte is an E4M3 NaN code
 * (0x7F, 0xFF; use lba_count_nan_codes to check), scales are finite and > 0.  Every zero
 * produced by the chain is +0.
 */
#ifndef LBA_H_
#define LBA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Q^FLOAT_{M,E,b} of Eq. 2. */
typedef struct {
  int32_t man_bits; /* M, 1..23                                                             */
  int32_t exp_bits; /* E, 1..8: binades [-b, 2^E-b-1], none reserved                        */
  int32_t bias;     /* b, -96..192                                                          */
  int32_t rounding; /* LBA_ROUND_FLOOR (the paper's, Sec. 3) or LBA_ROUND_NEAREST_EVEN      */
  int32_t flags;    /* bit0 LBA_FLAG_UNDERFLOW: 1 = flush |x| < R_UF to 0 (Eq. 2);
                       0 = "excluding underflow" (first fine-tuning stage, Sec. 3);
                       bit2 LBA_FLAG_INPUT_M4E3, read from prod_fmt only: see below          */
} lba_fmt;

enum { LBA_ROUND_FLOOR = 0, LBA_ROUND_NEAREST_EVEN = 1 };
enum { LBA_FLAG_UNDERFLOW = 1, LBA_FLAG_WRAP = 2, LBA_FLAG_INPUT_M4E3 = 4 };

/* Input byte format.  By default both operands are OCP E4M3 bytes.  With LBA_FLAG_INPUT_M4E3 set in
 * prod_fmt->flags (the format of the multiplier, whose inputs these are) both operands are bytes of the paper's own
 * weight/activation format instead (Sec. 3.1: "M4E3 representation with flex-bias"): s eee mmmm, one sign bit,
 * 3 exponent bits, 4 mantissa bits, decoded as Eq. 2 gives for (M, E, b) = (4, 3, 0):
 *     value = (-1)^s * 2^e * (1 + m/16),  e = 0..7,  largest magnitude 248 = R_OF,
 * except that the code with e = m = 0 (0x00, 0x80) is zero: Eq. 2 has no code for zero, and this reading gives up
 * the magnitude 2^0 for it.  All 256 codes are numbers (no NaN).  The per-tensor flex-bias of Sec. 3.1, a power of
 * two, is the caller's scale_a / scale_b (per tensor), applied to the finished sum like every scale.  Products of
 * two such values carry up to 10 significant bits, so a product format with M < 9 cuts them (Q_prod of Eq. 4 acts
 * on the mantissa, which it never does for E4M3 inputs with M >= 7).  lba_gemm, lba_gemm_batched, lba_conv2d and the
 * host-buffer variants accept the flag with the floating-point quantisers of Eq. 2; the fixed-point formats and the
 * straight-through-estimator entry points return LBA_ERR_FORMAT for it. */

/* exp_bits = 0 selects the fixed-point quantiser Q^FIXED_{B,b} of Eq. 1 (Sec. 2.1) instead, for both formats of a
 * call or for neither (else LBA_ERR_FORMAT): man_bits = B, the number of bits including the sign, 2..24; bias = b
 * (product format: -64..12, accumulator: -64..64); rounding must be LBA_ROUND_FLOOR, which here is floor toward
 * minus infinity: Q(v) = 2^-b floor(v 2^b), held to [R_min, R_max] = [-2^(B-1), 2^(B-1) - 1] 2^-b by saturation as
 * in Eq. 1 or, with flags bit1 LBA_FLAG_WRAP, by two's-complement wrap-around (the integer accumulators that
 * Sec. 2.2 cites).  lba_gemm, lba_gemm_batched, lba_conv2d and the host-buffer variants accept such formats (an
 * integer-only inner loop); the straight-through-estimator entry points do not. */
enum { LBA_ORDER_SEQUENTIAL = 0, LBA_ORDER_CHUNKED = 1 };

enum {
  LBA_OK = 0,
  LBA_ERR_NULL = -1,      /* a required pointer is NULL                                      */
  LBA_ERR_SHAPE = -2,     /* a negative size, an empty convolution output, sizes beyond int32
                             where the kernel indexes with int32                             */
  LBA_ERR_FORMAT = -3,    /* M/E/b/rounding out of range, or a format whose reachable values
                             cannot be carried exactly in binary32 registers                 */
  LBA_ERR_ORDER = -4,     /* unknown order, or chunk < 1 in chunked order                    */
  LBA_ERR_SCALE_LEN = -5, /* a scale length that is neither 1 nor the matching dimension     */
  LBA_ERR_CUDA = -6,      /* a CUDA call failed; see lba_last_cuda_error                     */
  LBA_ERR_WORKSPACE = -7, /* host-buffer entry points: workspace NULL, too small, misaligned */
  LBA_ERR_STATIC_LIMIT = -8 /* lba_gemm_host_static: the problem needs more than LBA_STATIC_WORKSPACE_BYTES */
};

/* GEMM  out[m][n] = epilogue( dot(A[m][:], B[n][:]) ), i.e. Y = X W^T with x_i = X_mi,
 * w_i = W_ni (App. A).
 *   A        device, [M][K] E4M3 bytes, K contiguous
 *   B        device, [N][K] E4M3 bytes, K contiguous
 *   scale_a  device, 1 value (per tensor) or M values (per row); scale_a_len says which
 *   scale_b  device, 1 value or N values (per output channel)
 *   bias     device, N values, or NULL
 *   out      device, [M][N] binary32, row-major; out = fl(fl(y*scale_a)*scale_b) (+ bias)
 * 16-byte aligned A and B with K a multiple of 16 take the vector-load path; anything else
 * is accepted and takes a slower byte-wise loader with identical results.
 * M, N or K equal to 0 are legal (K = 0 gives y = 0).  Returns LBA_OK or a negative code;
 * on error nothing is enqueued. */
int lba_gemm(const uint8_t* A, const uint8_t* B, const float* scale_a, int scale_a_len, const float* scale_b,
             int scale_b_len, const float* bias, int64_t M, int64_t N, int64_t K, const lba_fmt* prod_fmt,
             const lba_fmt* acc_fmt, int order, int chunk, float* out, void* stream);

/* Batched GEMM: `batch` independent problems of the same shape and formats in one launch, problem z reading
 * A + z*stride_a and B + z*stride_b (byte offsets; [M][K] and [N][K] each) and writing out + z*stride_out
 * (offset in floats; [M][N]).  This is the matrix product inside attention (Q K^T and P V), which the paper
 * also routes through the LBA GEMM (App. C.2: all fully connected layers and matrix multiplications).
 * A stride of 0 shares that operand between all problems; otherwise strides must be at least one problem's
 * size, and stride_out always.  Scales and bias are shared by all problems (same lengths as lba_gemm).
 * Strides that are multiples of 16 keep the vector-load path. */
int lba_gemm_batched(const uint8_t* A, const uint8_t* B, const float* scale_a, int scale_a_len, const float* scale_b,
                     int scale_b_len, const float* bias, int64_t batch, int64_t M, int64_t N, int64_t K,
                     int64_t stride_a, int64_t stride_b, int64_t stride_out, const lba_fmt* prod_fmt,
                     const lba_fmt* acc_fmt, int order, int chunk, float* out, void* stream);

/* Re-computation for the recursive overflow straight-through estimator (Sec. 4 and App. D): the forward pass is
 * deterministic, so the backward pass can replay it instead of storing one bit per FMAq.  For every output
 * (m, n), in SEQUENTIAL order, last[m][n] is the largest step index i with
 *     | Q_prod(x_i w_i) + S_i | >= R_OF(acc_fmt)        (STE^OF = 0 at that step),
 * or -1 if the accumulator never overflowed: the recursive estimator cuts the gradient of every product before
 * that step and passes the later ones, so this index is all it needs per output (App. D).
 *   A, B   device, as for lba_gemm; formats must use floor rounding (else LBA_ERR_FORMAT)
 *   last   device, [M][N] int32 */
int lba_gemm_last_overflow(const uint8_t* A, const uint8_t* B, int64_t M, int64_t N, int64_t K, const lba_fmt* prod_fmt,
                           const lba_fmt* acc_fmt, int32_t* last, void* stream);

/* Straight-through estimators of App. D, per FMAq step. */
enum { LBA_STE_OF = 1, LBA_STE_DIFF = 2 };

/* Re-computation for the fine-grained estimators (Sec. 4, App. D): replays the chain of every output (m, n) in the
 * given order and writes one bit per FMAq step, 1 where the estimator passes the gradient:
 *   LBA_STE_OF    1 iff | Q_prod(x_i w_i) + S_i | < R_OF(acc_fmt)
 *   LBA_STE_DIFF  1 iff | FMAq(x_i, w_i, S_i) - S_i | > eps2 * ( |x_i w_i| + eps1 ), evaluated in binary32 with one
 *                 rounding (to nearest) per operation: the subtraction, the addition, the multiplication;
 *                 eps1, eps2 > 0 are given in the domain of the decoded code values (the paper does not print
 *                 the values it used).
 * mask1 [M][ceil(K/32)][N] uint32 (the words of one step range lie side by side for neighbouring n, which is how
 * both this kernel and a gradient GEMM that reduces over n touch them): bit (i % 32) of word (i / 32) of output
 * (m, n) belongs to step i of the first hierarchy (the only one in sequential order).  In chunked order
 * mask2 [M][ceil(C/32)][N], C = ceil(K/chunk), holds in the same way the
 * bits of the steps T <- Q_acc(C_j + T) that fold chunk j into the second hierarchy, with the chunk sum C_j in the
 * product's place; a single chunk (chunk >= K) still has its one fold.  Unused high bits of a last word are 0.
 * The "immediate" estimators use the bits as they are; the "recursive" ones pass a product's gradient only if every
 * later step on its path to the output passed, which the caller derives from the same bits (App. D).
 *   A, B          device, as for lba_gemm; floor rounding only (else LBA_ERR_FORMAT)
 *   ste           LBA_STE_OF or LBA_STE_DIFF (else LBA_ERR_ORDER); eps1, eps2 are read for LBA_STE_DIFF only, and
 *                 values for which the comparison cannot be carried in binary32 give LBA_ERR_FORMAT
 *   mask1, mask2  device, written in full by the call; mask2 may be NULL in sequential order */
int lba_gemm_ste_mask(const uint8_t* A, const uint8_t* B, int64_t M, int64_t N, int64_t K, const lba_fmt* prod_fmt,
                      const lba_fmt* acc_fmt, int order, int chunk, int ste, float eps1, float eps2, uint32_t* mask1,
                      uint32_t* mask2, void* stream);

/* Convolution as an implicit GEMM (Eq. 3 with m = (b, oh, ow), n = c_out and k walking
 * (kh, kw, c_in), c_in fastest).  Padded taps are the value 0 and still count toward the
 * chunk position.  Dilation 1, groups 1.
 *   x        device, [B][H][W][C_in] E4M3 bytes (NHWC)
 *   w        device, [C_out][KH][KW][C_in] E4M3 bytes
 *   scale_x  device, 1 value or B*H_out*W_out values; scale_w: 1 or C_out values
 *   bias     device, C_out values, or NULL
 *   out      device, [B][H_out][W_out][C_out] binary32,
 *            H_out = (H + 2*pad_h - KH)/stride_h + 1, likewise W_out
 * C_in a multiple of 16 with 16-byte aligned x and w takes the vector-load path. */
int lba_conv2d(const uint8_t* x, const uint8_t* w, const float* scale_x, int scale_x_len, const float* scale_w,
               int scale_w_len, const float* bias, int B, int H, int W, int C_in, int C_out, int KH, int KW,
               int stride_h, int stride_w, int pad_h, int pad_w, const lba_fmt* prod_fmt, const lba_fmt* acc_fmt,
               int order, int chunk, float* out, void* stream);

/* The same two operations on HOST buffers (pinned memory recommended): inputs are copied to
 * the caller's device workspace, the kernel runs, and `out` (host) receives the result; all
 * of it is enqueued on `stream`, so the caller synchronises the stream before reading `out`.
 * `workspace` is device memory, 256-byte aligned, of at least lba_*_host_workspace_bytes(...)
 * bytes; the library does not allocate.  A shape whose operand or output byte counts do not fit
 * in 62 bits is refused (the size functions return 0, the calls LBA_ERR_SHAPE) before anything
 * is copied. */
size_t lba_gemm_host_workspace_bytes(int64_t M, int64_t N, int64_t K, int scale_a_len, int scale_b_len,
                                     int has_bias);
int lba_gemm_host(const uint8_t* A, const uint8_t* B, const float* scale_a, int scale_a_len, const float* scale_b,
                  int scale_b_len, const float* bias, int64_t M, int64_t N, int64_t K, const lba_fmt* prod_fmt,
                  const lba_fmt* acc_fmt, int order, int chunk, float* out, void* workspace,
                  size_t workspace_bytes, void* stream);
size_t lba_conv2d_host_workspace_bytes(int B, int H, int W, int C_in, int C_out, int KH, int KW, int stride_h,
                                       int stride_w, int pad_h, int pad_w, int scale_x_len, int scale_w_len,
                                       int has_bias);
int lba_conv2d_host(const uint8_t* x, const uint8_t* w, const float* scale_x, int scale_x_len,
                    const float* scale_w, int scale_w_len, const float* bias, int B, int H, int W, int C_in,
                    int C_out, int KH, int KW, int stride_h, int stride_w, int pad_h, int pad_w,
                    const lba_fmt* prod_fmt, const lba_fmt* acc_fmt, int order, int chunk, float* out,
                    void* workspace, size_t workspace_bytes, void* stream);

/* lba_gemm_host for callers that must not allocate device memory.  (No counterpart in the paper: it
 * is a packaging variant of lba_gemm_host, computing exactly the same result.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a region whose device memory
 * is budgeted and handed out up front (an inference server's arena, a plug-in that was given no
 * allocator), in a callback or a latency-critical loop where an allocation would synchronise the
 * device, or after start-up in a process that has promised not to grow its footprint.  lba_gemm_host
 * asks such a caller for a device workspace it has no way to obtain; this entry point brings its own.
 *
 * The workspace is a fixed array of LBA_STATIC_WORKSPACE_BYTES bytes that is part of the library
 * image: every GPU on which the library is loaded holds that much memory from load until the process
 * exits, whether or not this function is ever called.  Arguments are those of lba_gemm_host without
 * the workspace pair; A, B, scales, bias and out are HOST buffers, copied on `stream`.
 *   - A problem with lba_gemm_host_workspace_bytes(...) > LBA_STATIC_WORKSPACE_BYTES is refused with
 *     LBA_ERR_STATIC_LIMIT and nothing is enqueued (roughly: M*K + N*K + 4*M*N must fit in 8 MiB).
 *   - The first call on each device looks up the array's device address (once, with that device
 *     current) and keeps it; make that first call outside any stream capture.  The kept address belongs
 *     to the device's primary context as it was then: after cudaDeviceReset (or anything else that
 *     destroys and re-creates that context) it is stale, and this entry point must not be used again
 *     in the same process.
 *   - All calls on a device share the one array, and it keeps whatever the previous call left there.
 *     Nothing in it has to start at zero: each call overwrites the operand areas it reads and the
 *     kernel writes every output element before it is copied back.  Two calls whose work overlaps on
 *     the GPU (different streams, or different host threads) race on the array: serialise them.
 *   - No cudaMalloc, cudaFree or other allocating call is made, on the first call or later. */
#define LBA_STATIC_WORKSPACE_BYTES (8u << 20)
int lba_gemm_host_static(const uint8_t* A, const uint8_t* B, const float* scale_a, int scale_a_len,
                         const float* scale_b, int scale_b_len, const float* bias, int64_t M, int64_t N, int64_t K,
                         const lba_fmt* prod_fmt, const lba_fmt* acc_fmt, int order, int chunk, float* out,
                         void* stream);

/* Debug helper for the NaN-code precondition: adds to *count (device, uint64, caller zeroes
 * it) the number of bytes among codes[0..n) equal to 0x7F or 0xFF. */
int lba_count_nan_codes(const uint8_t* codes, int64_t n, unsigned long long* count, void* stream);

/* Which kernel variant a call with these arguments would run, as text, e.g.
 * "tile=64x64x16 micro=4x8 q=floor_fast pq=none kernel=packed order=chunk16 load=gemm_vec grid=128x128"
 * (pq: what Q_prod does beyond its flush -- none, cut = mantissa cut, cut_sat = cut and saturation, fused = Q_prod is
 * the identity on every reachable product, so product and sum are one instruction; kernel: the
 * packed two-outputs-per-instruction kernel or the generic scalar one).
 * is_conv selects the loader family; for a convolution pass M = B*H_out*W_out, N = C_out,
 * K = KH*KW*C_in and vec_ok = (C_in % 16 == 0 and pointers aligned).  Returns LBA_OK or the
 * error the real call would return; buf may be NULL. */
int lba_describe_plan(int64_t M, int64_t N, int64_t K, const lba_fmt* prod_fmt, const lba_fmt* acc_fmt, int order,
                      int chunk, int is_conv, int vec_ok, char* buf, size_t buf_len);
/* The same for lba_gemm_batched with `batch` problems (batch >= 1, else LBA_ERR_SHAPE): the tile is chosen for the
 * CTAs of all problems together; the grid printed is that of one problem. */
int lba_describe_plan_batched(int64_t batch, int64_t M, int64_t N, int64_t K, const lba_fmt* prod_fmt,
                              const lba_fmt* acc_fmt, int order, int chunk, int is_conv, int vec_ok, char* buf,
                              size_t buf_len);

/* Testing and tuning hook: force the CTA tile (0 = 128x128, 1 = 128x64, 2 = 64x64, 3 = 32x32 outputs; 5 = the 64x64
 * tile shared by a cluster of two CTAs, each taking every second chunk, used only in chunk-16 order with floor
 * rounding and 16-byte loads, ignored otherwise; -1 = automatic choice, the default).  For lba_gemm_ste_mask, 3
 * selects the scalar tracking kernel where the packed one would run.  Results never depend on the tile, only speed
 * does.  The setting is one process-wide word (an atomic store): it is meant for tests and tuning runs, it applies
 * to every thread's later calls, and a caller that changes it while other threads are inside the library gets an
 * unspecified mix of old and new tiles, never a wrong result.  Returns LBA_OK, or LBA_ERR_SHAPE for an unknown tile. */
int lba_set_tile_override(int tile);

const char* lba_status_string(int status);
int lba_last_cuda_error(void); /* cudaError_t of the most recent failed CUDA call in this thread, else 0 */
int lba_version(void);

#ifdef __cplusplus
}
#endif
#endif /* LBA_H_ */
