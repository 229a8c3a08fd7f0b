/*
 * tdq.h -- C ABI of the COD-TDQ hot path on NVIDIA B200 (sm_100a).
 *
 * The library quantizes token activations with token-group scales (DSTG) whose clip
 * radius is projected by two bounds (DCRP), quantizes weights per output channel, and
 * runs the W4A4 linear layer on the 4-bit codes.
 *
 * Conventions shared by every call
 *   - Unless a parameter is marked HOST, pointers are DEVICE pointers owned by the caller.
 *     The library allocates nothing, frees nothing and keeps no pointer after the call.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL is the
 *     default stream) and the call returns without waiting for it.
 *   - Arguments are checked on the host before anything is launched.  A bad argument
 *     returns an error code and launches nothing.  Nothing throws, aborts or traps.
 *   - Kernels whose threads wait on each other give every wait a limit of about a second.  A
 *     wait that runs out records a code and the kernel returns with part of its output
 *     unwritten.  The linear-layer calls record it in the call's workspace, read back by
 *     tdq_workspace_status(); the quantizer calls, which have no workspace, in one word per
 *     device, read back (and cleared) by tdq_quantize_status().
 *   - The library allocates no device memory.  tdq_quant_linear_host creates two streams and
 *     a few events per device on first use and keeps them for the life of the process; no
 *     other call creates CUDA objects.
 *   - Non-finite inputs (NaN, Inf) give unspecified codes; they never fault.
 *
 * Notation (the paper's): M = B*N tokens, C = I input channels, O output channels,
 * g group size, K = C_pad / g groups per token with C_pad = g * ceil(C / g),
 * q_max = 7, q_min = -8.
 */
#ifndef TDQ_H_
#define TDQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    TDQ_OK = 0,
    TDQ_ERR_INVALID_ARG = 1,    /* null pointer, non-positive size, parameter out of range   */
    TDQ_ERR_UNSUPPORTED = 2,    /* a legal request this build has no kernel for              */
    TDQ_ERR_ALIGNMENT = 3,      /* a pointer or stride misses the alignment stated below     */
    TDQ_ERR_WORKSPACE = 4,      /* workspace missing or smaller than the size query returns  */
    TDQ_ERR_CUDA = 5,           /* a CUDA runtime or driver call failed                      */
    TDQ_ERR_DEVICE_TIMEOUT = 6  /* a bounded device-side wait ran out (see workspace status) */
} tdq_status;

typedef enum { TDQ_F32 = 0, TDQ_BF16 = 1, TDQ_F16 = 2 /* outputs of the linear layer only */ } tdq_dtype;

/* Which DCRP bounds take part in the projection (Algorithm S1 step 4; the ablation
 * variants of Table S6).  Both = COD-TDQ, neither = DSTG only. */
#define TDQ_ENABLE_C1 1u  /* step-to-dispersion bound, Eq. 10 */
#define TDQ_ENABLE_C2 2u  /* zero-bin mass bound, Eq. 11      */
/* A variant, not the paper's quantizer: after the projection the step is rounded DOWN to a power of
 * two, Delta' = 2^floor(log2 Delta), and c' = 7 Delta'.  Both DCRP bounds are upper bounds on c, so they
 * still hold; the clip range shrinks by up to a factor of two.  Such steps let tdq_w4a4_linear_pow2
 * fold the group scale into the tensor-core operand. */
#define TDQ_POW2_STEP 4u

typedef struct {
    int32_t group_size;      /* g, even, 2..4096; default 32.  g == C_pad gives one scale per token */
    float tau;               /* C1: Delta_k / sigma_k <= tau, tau > 0; default 1.0                   */
    float zr;                /* C2: zero-bin mass bound in (0,1]; default 0.2; rank ceil(zr*g)       */
    float base_percentile;   /* p in (0,1]; 1.0 = max-abs base radius, else rank ceil(p*g) (Eq. 6)   */
    uint32_t flags;          /* TDQ_ENABLE_C1 | TDQ_ENABLE_C2 [| TDQ_POW2_STEP]                      */
} tdq_act_params;

/* The paper's shared setting (g, tau, zr) = (32, 1.0, 0.2), max-abs base radius, both bounds. */
void tdq_default_act_params(tdq_act_params* p /* HOST, out */);

/*
 * Token-group dual-constraint activation quantizer: Algorithm S1 steps 1-7 (Eq. 5-12).
 * For every token m and channel group k:
 *   c_base = max |x| (or the ceil(p*g)-th smallest |x|);  sigma = population std + 1e-12;
 *   thr = ceil(zr*g)-th smallest |x|;  c = max(min(c_base, 7*tau*sigma, 14*thr), 1e-8);
 *   Delta = max(c/7, 1e-8);  q = clip(round_half_even(clip(x,-c,c) / Delta), -8, 7).
 * Channels C..C_pad-1 are zeros; they take part in the statistics and get code 0.
 *
 *   x          [B*N rows, C] row-major, x_dtype, consecutive rows row_stride_elems apart
 *              (>= C).  No alignment is required; 16-byte aligned x with C % 32 == 0,
 *              row_stride_elems % 8 == 0 and g == 32 takes the fast kernels, whatever the two
 *              ranks (the maximum as base radius with any zero-bin rank, and base ranks 29-31
 *              with zero-bin rank 7, have kernels of their own; any other pair runs a kernel
 *              that takes its ranks at run time, about a fifth slower); anything else takes a
 *              much slower general kernel with the same results.
 *   codes      [B*N, C_pad/2] bytes; byte j of a row holds channel 2j in its low nibble
 *              and channel 2j+1 in its high nibble, two's complement.
 *   scale      [B*N, K] float32, Delta_k.
 *   offset     NULL, or [B*N, K] float32 that is filled with 0 (the grid is symmetric:
 *              the paper's quantizer has no zero point).
 * Errors: TDQ_ERR_INVALID_ARG for null x/p/codes/scale, B,N < 0, C <= 0, stride < C, odd or
 * out-of-range g, tau <= 0, zr or p outside (0,1].  B*N == 0 is a no-op returning TDQ_OK.
 */
tdq_status tdq_quantize_act(const void* x, tdq_dtype x_dtype, int64_t B, int64_t N, int64_t C,
                            int64_t row_stride_elems, const tdq_act_params* p /* HOST */,
                            uint8_t* codes, float* scale, float* offset, void* cuda_stream);

/*
 * The same quantizer for channel-major input (the 4-D branch of Supp. S1.1, where a feature
 * map [B, C, H, W] is quantized along C): x is read in place, without the permuted copy that
 * tdq_quantize_act would need, and the outputs are token-major like tdq_quantize_act's with
 * token index (b*H + h)*W + w:   codes [B*H*W, C/2],  scale [B*H*W, C/32],  offset NULL or
 * [B*H*W, C/32].  They can go straight into tdq_w4a4_linear (a 1x1 convolution).
 *   x   [B, C, H, W] contiguous.  16-byte aligned x with H*W*sizeof(element) % 16 == 0 is read
 *       with vector loads, anything else element by element.
 * Fast path only: TDQ_ERR_UNSUPPORTED unless group_size == 32, C % 32 == 0, base_percentile
 * gives the maximum (rank 32), codes is 16-byte aligned and, with C2 on, ceil(32 zr) is one
 * of 4, 7, 10, 13, 16, 32; also if C/32 or B exceeds 65535.  Other errors as above.
 */
tdq_status tdq_quantize_act_nchw(const void* x, tdq_dtype x_dtype, int64_t B, int64_t C, int64_t H,
                                 int64_t W, const tdq_act_params* p /* HOST */, uint8_t* codes,
                                 float* scale, float* offset, void* cuda_stream);

/*
 * Fixed-radius control (the fixed offline-calibrated variant of Supp. S1.2 and S4.2): the clip
 * radius is a number chosen beforehand for the whole layer, so nothing is reduced over the
 * activations.  With c = max(radius, 1e-8) in every group:
 *   Delta = max(c/7, 1e-8);  q = clip(round_half_even(clip(x,-c,c) / Delta), -8, 7).
 *   x, B, N, C, row_stride_elems as for tdq_quantize_act;  codes [B*N, C/2];  scale [B*N, C/g]
 *   (every entry Delta, so that the outputs feed tdq_w4a4_linear unchanged);  offset NULL or
 *   [B*N, C/g], filled with 0.
 * TDQ_ERR_INVALID_ARG for null pointers, radius <= 0 or a bad group size; TDQ_ERR_UNSUPPORTED
 * unless group_size % 8 == 0, C % group_size == 0, x is 16-byte aligned with a row pitch that is
 * a multiple of 16 bytes, and codes is 4-byte aligned.
 */
tdq_status tdq_quantize_act_fixed(const void* x, tdq_dtype x_dtype, int64_t B, int64_t N, int64_t C,
                                  int64_t row_stride_elems, int32_t group_size, float radius,
                                  uint8_t* codes, float* scale, float* offset, void* cuda_stream);

/*
 * Static weight quantizer, Eq. 4 with absmax per-output-channel scales:
 *   s_o = max(max_i |W[o,i]| / 7, 1e-8);  Q = clip(round_half_even(W / s_o), -8, 7).
 *   w       [O, I] row-major, contiguous, w_dtype.
 *   pad_to  the input dimension is zero-padded to I_pad, a multiple of pad_to (even;
 *           pass the activation group size so both operands share C_pad).
 *   wcodes  [O, I_pad/2] bytes, nibble order as for activations.   wscale [O] float32.
 */
tdq_status tdq_quantize_weight(const void* w, tdq_dtype w_dtype, int64_t O, int64_t I, int32_t pad_to,
                               uint8_t* wcodes, float* wscale, void* cuda_stream);

/*
 * The affine mode of the auxiliary Linear I/O correction of Supp. S1.1 (modes none / bias / affine; the paper
 * names the modes without a formula, the reading taken here is a per-output-channel y' = a_o y + b_o applied to
 * the layer's output y = s_o Sigma + bias_o).  The correction is static, so it costs nothing at run time when it
 * is folded into the layer's constants once:  wscale_out[o] = a_o s_o,  bias_out[o] = a_o bias_o + b_o, each
 * rounded to binary32; tdq_w4a4_linear (or the fused call) with these two vectors then computes y'.  The result
 * differs from a_o (s_o Sigma + bias_o) + b_o evaluated exactly by a few units in the last place of its terms.
 *   wscale [O], bias NULL or [O], out_mul [O] (a_o), out_add NULL or [O] (b_o); wscale_out [O] and bias_out [O]
 *   may alias wscale and bias.  The bias mode of the correction is the bias vector of tdq_w4a4_linear itself.
 */
tdq_status tdq_fold_output_affine(const float* wscale, const float* bias, const float* out_mul, const float* out_add,
                                  int64_t O, float* wscale_out, float* bias_out, void* cuda_stream);

/*
 * W4A4 linear layer, Algorithm S1 step 10 with x_hat = Delta_k q (Eq. 9) and
 * W_hat = s_o Q_w (Eq. 4) substituted:
 *   acc[m,o,k] = sum_{i in group k} q_x[m,i] * q_w[o,i]            (exact, int32)
 *   y[m,o]     = s_o * sum_k Delta[m,k] * acc[m,o,k]  (+ bias[o])   (float32)
 *   xcodes [M, I_pad/2], xscale [M, K], wcodes [O, I_pad/2], wscale [O], bias NULL or [O].
 *   I_pad must be a multiple of group_size; group_size a multiple of 32 (the integer
 *   tensor-core instruction contracts 32 codes at a time), at most 4096.
 *   y      [M, O], y_dtype (float32, bf16 or fp16; the 16-bit types are rounded to nearest even from the
 *          float32 result), rows y_row_stride elements apart (>= O).
 *   acc_debug  NULL, or [M, O, K] int32 receiving every group's integer dot product
 *              (for tests; slows the kernel down).
 *   workspace  at least tdq_linear_workspace_bytes() bytes, 16-byte aligned.  Holds the
 *              status word read by tdq_workspace_status().  The call clears it first, so
 *              one workspace must not be shared by calls that overlap in time.
 * Alignment: xcodes, wcodes 16 bytes; I_pad/2 % 16 == 0 is implied by g % 32 == 0.
 */
tdq_status tdq_w4a4_linear(const uint8_t* xcodes, const float* xscale, const uint8_t* wcodes,
                           const float* wscale, const float* bias, int64_t M, int64_t I_pad, int64_t O,
                           int32_t group_size, void* y, tdq_dtype y_dtype, int64_t y_row_stride,
                           int32_t* acc_debug, void* workspace, size_t workspace_bytes,
                           void* cuda_stream);

/*
 * The linear layer for activations quantized with TDQ_POW2_STEP (a variant; the paper has no
 * counterpart).  When every step of a token is a power of two, Delta[m,k] = 2^(e_m + s[m,k]), the
 * group scale can ride inside the tensor-core operand: a code is stored as the FP8 (E4M3) value
 * q * 2^(s - 9), which is exact for s in 0..14, the whole contraction accumulates in one fp32
 * accumulator, and each row is scaled once, by 2^e_m * s_o, at the end.  There is no per-group pass
 * over the accumulators, which is what bounds tdq_w4a4_linear at g = 32.
 *   Arguments as for tdq_w4a4_linear (no acc_debug).  xscale entries must be positive powers of
 *   two; anything else is reported through tdq_workspace_status (detail code 11) and the output
 *   is then meaningless.
 *   e_m is the largest step exponent of the row minus 14.  Steps more than 2^14 below the row's
 *   largest lose low bits of their codes (truncation; the lost part is below 2^-14 of the row's
 *   largest step per element).  Sums are accumulated in binary32 by the tensor core, in its
 *   order: results agree with tdq_w4a4_linear on the same inputs to about 1e-6 relative to the sum
 *   of the absolute terms, not bit for bit.
 */
tdq_status tdq_w4a4_linear_pow2(const uint8_t* xcodes, const float* xscale, const uint8_t* wcodes,
                                const float* wscale, const float* bias, int64_t M, int64_t I_pad, int64_t O,
                                int32_t group_size, void* y, tdq_dtype y_dtype, int64_t y_row_stride,
                                void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Quantizer fused into the linear layer as the producer of its A operand (Algorithm S1 steps
 * 1-10 in one kernel, with no pass over the activations besides the layer's own): the same
 * result, bit for bit, as tdq_quantize_act followed by tdq_w4a4_linear, but activation codes
 * and scales never reach global memory.  For every block of 128 token rows the kernel
 * quantizes the rows into shared memory and keeps them there for all output columns.
 *   x, B, N, C, row_stride_elems, p   as for tdq_quantize_act;   wcodes [O, C/2], wscale [O],
 *   bias NULL or [O];   y, y_dtype, y_row_stride, workspace as for tdq_w4a4_linear
 *   (workspace size: tdq_linear_workspace_bytes(B*N, C, O, 32)).
 * TDQ_ERR_UNSUPPORTED unless: group_size == 32, C % 32 == 0, base_percentile == 1, x 16-byte
 * aligned with a row pitch that is a multiple of 16 bytes, the zero-bin rank ceil(32 zr) == 7
 * when the C2 bound is enabled, and C <= 768 (a row block's operand bytes must fit in shared
 * memory).  Callers fall back to the two calls in those cases.
 * Speed: on the benchmark workloads this call is not faster than the two calls it replaces (a tie on the
 * smallest, about a third slower on the largest); its use is that activation codes never reach memory.
 */
tdq_status tdq_quant_linear_fused(const void* x, tdq_dtype x_dtype, int64_t B, int64_t N, int64_t C,
                                  int64_t row_stride_elems, const tdq_act_params* p /* HOST */,
                                  const uint8_t* wcodes, const float* wscale, const float* bias,
                                  int64_t O, void* y, tdq_dtype y_dtype, int64_t y_row_stride,
                                  void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The two-kernel path with HOST input and output: copies x_host to x_dev, runs
 * tdq_quantize_act and tdq_w4a4_linear, copies y_dev to y_host.  The rows go through in up to
 * eight chunks: the kernels run on cuda_stream, the copies on two side streams of the library
 * (created on the first call on a device and tied to cuda_stream by events), so that the
 * copy-out of one chunk overlaps the copy-in and the kernels of the next.  Work queued on
 * cuda_stream after the call starts only when the last copy-out has finished.
 * x_host / y_host should be page-locked for the copies to be asynchronous.  The device
 * buffers are the caller's and sized as for the two calls (x_dev [B*N, C] dense).  The chunks
 * share the workspace one after another, so tdq_workspace_status afterwards speaks for the last
 * chunk only.  Not for concurrent use from several host threads on one device.
 */
tdq_status tdq_quant_linear_host(const void* x_host /* HOST */, tdq_dtype x_dtype, int64_t B, int64_t N,
                                 int64_t C, const tdq_act_params* p /* HOST */, const uint8_t* wcodes,
                                 const float* wscale, const float* bias, int64_t O,
                                 void* y_host /* HOST */, tdq_dtype y_dtype,
                                 void* x_dev, uint8_t* codes_dev, float* scale_dev, void* y_dev,
                                 void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * tdq_w4a4_linear for callers that cannot allocate device memory.  (An addition of this library:
 * the paper has no counterpart.)  Some code that wants to run the linear layer has no way to
 * obtain a workspace: a plug-in running inside a host application that owns all device memory,
 * a callback where calling cudaMalloc is forbidden or would synchronise the whole device, a
 * process whose memory budget was handed out up front.  This entry point computes exactly what
 * tdq_w4a4_linear computes, with the same argument meaning and checks, but keeps the operand
 * blocks and the status word in an array that is part of the library image itself
 * (TDQ_LINEAR_STATIC_BYTES, 8 MiB, in every CUDA context that loads the library,
 * from load until the process exits).  It calls no allocating or freeing routine.
 *   - Problems whose tdq_linear_workspace_bytes() exceed the capacity are refused with
 *     TDQ_ERR_WORKSPACE and nothing is launched (of the five benchmark workloads the first
 *     three fit).  There is no acc_debug output.
 *   - The first call on each device, made with that device current, looks up where the array
 *     lives on that device; make that first call outside any stream capture.
 *   - All calls share the one array, which keeps whatever the last call left in it.  Every call
 *     rewrites all the blocks it is going to read and clears the status word, so earlier
 *     contents never leak into a result; but two calls that overlap on the GPU (different
 *     streams, or different host threads) race on it.  Order them on one stream.
 *   - wait != 0: the call returns only after its work on cuda_stream has finished, and answers
 *     TDQ_ERR_DEVICE_TIMEOUT if a bounded wait inside the kernel ran out.  wait == 0: the call
 *     is asynchronous like tdq_w4a4_linear and that condition goes unreported.
 */
#define TDQ_LINEAR_STATIC_BYTES ((size_t)8 << 20)
tdq_status tdq_w4a4_linear_static(const uint8_t* xcodes, const float* xscale, const uint8_t* wcodes,
                                  const float* wscale, const float* bias, int64_t M, int64_t I_pad, int64_t O,
                                  int32_t group_size, void* y, tdq_dtype y_dtype, int64_t y_row_stride,
                                  int32_t wait, void* cuda_stream);

/* Bytes of workspace tdq_w4a4_linear / tdq_quant_linear_fused need for this problem. */
size_t tdq_linear_workspace_bytes(int64_t M, int64_t I_pad, int64_t O, int32_t group_size);

/*
 * Waits for cuda_stream, then reads the status word a linear call left in its workspace:
 * TDQ_OK, or TDQ_ERR_DEVICE_TIMEOUT when a bounded wait inside the kernel ran out (the
 * output of that call is then incomplete).  detail (HOST, nullable) receives the raw word:
 * bits 0-7 name the wait that gave up, bits 8-31 the tile index.
 */
tdq_status tdq_workspace_status(const void* workspace, void* cuda_stream, uint32_t* detail /* HOST */);

/*
 * Waits for cuda_stream, then reads the word in which the quantizer kernels of the current device
 * (tdq_quantize_act and its variants, which have no workspace) record a bounded wait that ran out:
 * TDQ_OK, or TDQ_ERR_DEVICE_TIMEOUT when one did since the last query (codes and scales of that
 * call are then incomplete).  detail (HOST, nullable) receives the raw word: bits 0-7 name the wait
 * (12 the tile producer, 13 a consumer warp, 14 the self-test), bits 8-31 the thread block.  A
 * non-zero word is cleared by the query.  The word is shared by all streams of the device.
 */
tdq_status tdq_quantize_status(void* cuda_stream, uint32_t* detail /* HOST */);

/*
 * Self-test of the bounded waits (no counterpart in the paper): one warp waits, with the kernels' own
 * wait routine and a limit of limit_cycles SM clocks (1000 .. 2e9), on a barrier that nobody arrives
 * on, gives up, records its code and returns; no copy or tensor-core operation is in flight when it
 * leaves, so the device stays usable.
 *   which == 0: the linear layer's routine; the code (15) goes to the status word of `workspace`
 *               (16-byte aligned, at least 256 bytes), which the call clears first; read it with
 *               tdq_workspace_status().
 *   which == 1: the quantizer's routine; the code (14) goes to the per-device word that
 *               tdq_quantize_status() reads; workspace is ignored.
 * The call is asynchronous on cuda_stream like every other one.
 */
tdq_status tdq_selftest_wait_timeout(int32_t which, int64_t limit_cycles, void* workspace, void* cuda_stream);

/*
 * Measures how fast the tensor cores of the current device run the instruction the linear layer is built on (no
 * counterpart in the paper; the benchmark uses it for its own dense 8-bit peak): one thread block per SM issues
 * n_mma tcgen05.mma instructions of shape 128 x 128 x 32 on operands resident in shared memory, with nothing else
 * running, and the slowest SM's clocks per instruction come back in *clocks_per_mma (HOST).  Peak operations per
 * second = 2 * 128 * 128 * 32 * SMs * SM clock / clocks_per_mma.
 *   integer_kind  0: E4M3 operands, float32 accumulator (the g = 32 route); 1: int8 operands, int32 accumulator.
 *   n_mma         a multiple of 4 between 4 and 2^22.
 *   scratch       device memory, 16-byte aligned, at least 16 bytes per SM.
 * The call waits for its kernel (it is a measurement, not part of the path).
 */
tdq_status tdq_measure_mma_clocks(int32_t integer_kind, int32_t n_mma, void* scratch, size_t scratch_bytes,
                                  double* clocks_per_mma /* HOST */, void* cuda_stream);

/* Static description of a status code. */
const char* tdq_status_string(tdq_status s);

/* Number of kernels this library has launched in the calling process (for accounting). */
uint64_t tdq_kernel_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* TDQ_H_ */
