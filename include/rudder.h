/*
 * rudder.h -- C ABI of the B200 (sm_100a) implementation of the SteerQuant / Rudder inference hot
 * path: the quantized linear layer of a world-action-model diffusion Transformer.
 *
 * One weight matrix per layer is quantised offline to 4 bits with the shared channel scaling D
 * folded in (Eq. 6; Section 4.2, last paragraph) and then serves every token stream and every
 * denoising step.  At run time a first kernel applies D^-1 and the per-stream, per-step gain
 * gamma on the fly while quantising the activations, and writes only the codes Q_X and one row
 * scale r_i (Section 4.4, first kernel; Eq. 8); a second kernel runs the low-bit GEMM and fuses
 * dequantisation, inverse-gain compensation and bias in its epilogue (Section 4.4, Eq. 10).
 *
 * General rules
 *   - Every pointer is a DEVICE pointer unless its comment says HOST.
 *   - The caller owns every buffer it passes (inputs, outputs, workspace).  The library owns only
 *     the memory inside a rudder_weight, allocated by rudder_pack_weights and released by
 *     rudder_weight_free.
 *   - Calls enqueue work on the given CUDA stream (a cudaStream_t passed as void*; NULL = the
 *     default stream) and return without synchronising, except where stated.  rudder_linear,
 *     rudder_block and rudder_quantize_activations allocate nothing.
 *   - Argument errors are detected on the host before anything is launched; nothing traps.
 *   - Device-side waits are bounded: a kernel that gives up records RUDDER_ERR_TIMEOUT in a device
 *     status word that rudder_device_status reads.
 *   - bf16 / fp16 values are passed as their 16-bit patterns (uint16_t).
 *   - Non-finite inputs are undefined behaviour (not checked).
 *   - A rudder_weight belongs to the device that was current when it was packed or imported.  Every call
 *     that takes one must be made with that device current and with buffers of that device; a call made
 *     with another device current returns RUDDER_ERR_ARG before anything is launched.
 *   - Host threads may call concurrently on different streams as long as they share no workspace;
 *     per-device state that is created on first use is guarded inside the library.
 *
 * Shapes: X is [M, K] row-major with leading dimension ldx (elements), W is [N, K] row-major (K
 * contiguous: the transpose of the paper's W in Y = X W), Y is [M, N] with leading dimension ldy.
 * K % 128 == 0, N % 64 == 0, M >= 1.  X, Y 16-byte aligned, ldx % 8 == 0, ldy % 8 == 0.
 */
#ifndef RUDDER_H
#define RUDDER_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    RUDDER_OK = 0,
    RUDDER_ERR_ARG = 1,          /* NULL required pointer, step outside [0,T), bad segments / stream id */
    RUDDER_ERR_SHAPE = 2,        /* unsupported M / N / K / group */
    RUDDER_ERR_ALIGN = 3,        /* pointer or leading dimension alignment */
    RUDDER_ERR_UNSUPPORTED = 4,  /* scheme / mode combination not available */
    RUDDER_ERR_WORKSPACE = 5,    /* workspace NULL, misaligned or too small */
    RUDDER_ERR_CUDA = 6,         /* a CUDA runtime / driver call failed */
    RUDDER_ERR_TIMEOUT = 7       /* a bounded device-side wait gave up */
} rudder_status;

/* Activation / weight number formats.  Weights are always 4-bit. */
typedef enum {
    RUDDER_W4A8_INT = 0,    /* INT4 weights (group scales), INT8 activations, q_max = 127 (Eq. 1, k = 8) */
    RUDDER_W4A4_INT = 1,    /* INT4 weights, INT4 activations, q_max = 7 (Eq. 1, k = 4); 8-bit tensor-core path
                               (integer MMA, or its exact E4M3 / FP32-accumulator form when group <= 128:
                               same integers, same results) */
    RUDDER_W4A4_NVFP4 = 2   /* E2M1 codes with a UE4M3 scale per 16 elements and an fp32 outer scale */
} rudder_scheme;

/* How the activation range a_i of Eq. 1 (c = a_i) is chosen. */
typedef enum {
    RUDDER_RANGE_PER_TOKEN = 0,  /* a_i = max_k |v_ik| of the scaled row */
    RUDDER_RANGE_STATIC = 1      /* a_i = clip[step]: the paper's calibrated threshold c_tau shared by all streams */
} rudder_range_mode;

typedef struct rudder_weight rudder_weight;   /* opaque; library-owned device memory */

/* Layer-step lookup table of calibrated gains and thresholds (Section 4.3, last paragraph). */
typedef struct {
    const float* gamma;      /* [T, S] gains gamma_{tau,s} > 0 */
    const float* clip;       /* [T] thresholds c_tau > 0, or NULL (required for RUDDER_RANGE_STATIC) */
    int T;                   /* denoising steps */
    int S;                   /* streams, 1..16 */
    rudder_range_mode mode;
} rudder_scale_table;

/* Row -> stream map s(i): contiguous segments of rows. */
typedef struct {
    const int32_t* seg_offsets;  /* HOST [n_seg + 1], ascending, seg_offsets[0] = 0, seg_offsets[n_seg] = M */
    const int32_t* seg_stream;   /* HOST [n_seg], each in [0, S) */
    int n_seg;                   /* 1..64 */
} rudder_segments;

/* ---------------------------------------------------------------------------------------------
 * rudder_pack_weights -- offline fold + quantise + pack (Eq. 6; Section 4.2 last paragraph; Eq. 1
 * with k = 4).  V = W diag(d); integer schemes: per (row j, group g of `group` input channels)
 * Delta_W[j,g] = fp16(max|V| / 7), codes = clip(round(V / Delta_W), -7, 7); NVFP4: tensor scale
 * max|V| / 2688, UE4M3 scale per 16 elements, E2M1 codes.  Also keeps dinv = 1 / d for the
 * run-time prologue.
 *   W [N,K] fp32, d [K] fp32 or NULL (= ones).  group: 64, 128 or K (K = the paper's per-output-
 *   channel scales); ignored for NVFP4.  Allocates the handle (cudaMalloc) and SYNCHRONISES the
 *   stream before returning.  *out is NULL on error.
 */
rudder_status rudder_pack_weights(const float* W, const float* d, int N, int K, rudder_scheme scheme,
                                  int group, void* stream, rudder_weight** out);
rudder_status rudder_weight_free(rudder_weight* w);

/* Shape and storage of a packed weight (HOST outputs; any may be NULL). */
rudder_status rudder_weight_info(const rudder_weight* w, int* N, int* K, int* group, int* scheme,
                                 size_t* device_bytes);

/* Canonical (layout-independent) view of a packed weight, for parity checks and storage:
 *   codes  uint8 [N, K/2]: low nibble = even k; INT4 two's complement, or E2M1 (bit 3 = sign)
 *   scales integer schemes: fp16 bit patterns [N, K/group]; NVFP4: UE4M3 bytes [N, K/16]
 *   dinv   fp32 [K];  tensor_scale fp32 [1] (NVFP4; 1.0 otherwise).  Any output may be NULL. */
rudder_status rudder_weight_export(const rudder_weight* w, uint8_t* codes, void* scales, float* dinv,
                                   float* tensor_scale, void* stream);

/* The inverse of rudder_weight_export: builds a packed weight from its canonical view ("stored as packed
 * integers with corresponding quantization scales", Section 4.2, last paragraph), e.g. from a checkpoint
 * written earlier.  Same layouts as above, all DEVICE pointers; tensor_scale is required for NVFP4 and
 * ignored otherwise; group as in rudder_pack_weights.  The handle behaves exactly like the one
 * rudder_pack_weights returned for the exported weight (same bits out of every kernel).  Allocates and
 * SYNCHRONISES the stream, like rudder_pack_weights. */
rudder_status rudder_weight_import(const uint8_t* codes, const void* scales, const float* dinv, const float* tensor_scale,
                                   int N, int K, rudder_scheme scheme, int group, void* stream, rudder_weight** out);

/* ---------------------------------------------------------------------------------------------
 * rudder_linear -- one quantized linear layer for one denoising step (Section 4.4; Eq. 8; Eq. 10):
 *   v_ik = (x_ik * dinv_k) * gamma[step, s(i)];  codes = clip(round(v * q_max / a_i));
 *   r_i = (a_i / q_max) / gamma;  C^(g) = codes . W-codes per weight group (INT32);
 *   Y_ij = bf16( (sum_g fp32(C^(g)_ij) Delta_W[j,g]) * r_i + b_j )      [group = K: exactly Eq. 10]
 * X bf16 [M, ldx], Y bf16 [M, ldy], bias fp32 [N] or NULL.  workspace holds Q_X and r between the
 * two kernels: at least rudder_linear_workspace_bytes(w, M) bytes, 256-byte aligned.
 */
size_t rudder_linear_workspace_bytes(const rudder_weight* w, int M);
rudder_status rudder_linear(const rudder_weight* w, const uint16_t* X, int64_t ldx, int M,
                            const rudder_segments* seg, int step, const rudder_scale_table* tab,
                            const float* bias, uint16_t* Y, int64_t ldy,
                            void* workspace, size_t workspace_bytes, void* stream);

/* rudder_linear_static -- rudder_linear without a caller-supplied workspace.  (The paper has no
 * counterpart: this is a convenience of this library.)
 * For callers that cannot allocate device memory -- code inside a captured or real-time region where
 * cudaMalloc is off limits, plug-ins that only receive input and output buffers, hosts whose memory
 * pool belongs to another component.  Q_X and r are kept in a fixed array of
 * rudder_linear_static_max_workspace_bytes() = 4 MiB that is part of the library image (every GPU
 * that loads the library holds it until the process exits).  The call allocates nothing.
 *   - Same arguments, results and errors as rudder_linear, minus the workspace.  If
 *     rudder_linear_workspace_bytes(w, M) exceeds the 4 MiB array the call returns
 *     RUDDER_ERR_WORKSPACE and launches nothing.
 *   - The first call on each device looks up the array's device address (with that device current);
 *     make that first call before any stream capture begins.
 *   - All calls on a device share the one array, which keeps the previous call's contents; nothing
 *     in it needs clearing between calls.  Two calls whose kernels may overlap on the GPU (different
 *     streams, or concurrent host threads) race on it: serialise them. */
size_t rudder_linear_static_max_workspace_bytes(void);
rudder_status rudder_linear_static(const rudder_weight* w, const uint16_t* X, int64_t ldx, int M,
                                   const rudder_segments* seg, int step, const rudder_scale_table* tab,
                                   const float* bias, uint16_t* Y, int64_t ldy, void* stream);

/* ---------------------------------------------------------------------------------------------
 * rudder_block -- the four quantized linears of one DiT block for one denoising step, replaying
 * caller-supplied inputs (the paper times DiT replay with captured inputs; attention, norms and
 * GELU stay in BF16 outside this library -- Appendix "Quantization" / "Efficiency").
 * Index 0..3 = QKV (H -> 3H), O (H -> H), MLP up (H -> F), MLP down (F -> H).
 */
typedef struct {
    const rudder_weight* w[4];
    const rudder_scale_table* tab[4];
    const float* bias[4];        /* each [N_l] or NULL */
    const uint16_t* x[4];        /* replay inputs, bf16 [M, ldx[l]]; x[1..3] may be NULL: chained (see below) */
    int64_t ldx[4];
    uint16_t* y[4];              /* outputs, bf16 [M, ldy[l]] */
    int64_t ldy[4];
} rudder_block_args;

/* Chained layers.  x[l] == NULL for l = 1, 2 or 3 makes that layer read the previous layer's output
 * through the minimal BF16 glue, so that the block runs end to end on the device from x[0] alone:
 *   O    (l = 1): the V third of the QKV output, y[0][:, 2 K_1 .. 3 K_1) -- a stand-in for attention, which
 *                 stays outside this library; requires N_0 == 3 K_1;
 *   up   (l = 2): the O output as it is (no norm / residual); requires N_1 == K_2;
 *   down (l = 3): rudder_gelu of the up output, staged at the end of the workspace; requires N_2 == K_3.
 *                 When the down projection's table has a static range (RUDDER_RANGE_STATIC: the paper's calibrated
 *                 threshold, Section 4.3) and an integer scheme, the GELU is applied INSIDE its prologue: with a_i = c_tau
 *                 the requantisation needs no row reduction, so one elementwise pass reads the up output, applies
 *                 the GELU and writes Q_X and r directly; the activated tensor is never stored (same bits either way).
 * A shape that does not chain returns RUDDER_ERR_SHAPE.  rudder_block_workspace_bytes accounts for the
 * staged GELU output (M x K_3 bf16) when x[3] is NULL.  rudder_block_host takes no NULL inputs. */
size_t rudder_block_workspace_bytes(const rudder_block_args* args, int M);
rudder_status rudder_block(const rudder_block_args* args, int M, const rudder_segments* seg, int step,
                           void* workspace, size_t workspace_bytes, void* stream);

/* rudder_block_dit -- the same four linears wired as one DiT block with its BF16 glue (normalisation, GELU and
 * residual additions stay in BF16: Appendix "Quantization"), run end to end on the device from x[0] alone:
 *     h   = x + O( V-third of QKV( rmsnorm(x; norm1_weight) ) )      [the V third stands in for attention, which stays outside]
 *     out = h + down( gelu( up( rmsnorm(h; norm2_weight) ) ) )
 * args->x[0] is the block input [M, H]; args->x[1..3] must be NULL; args->y[l] still receive the four linears' outputs;
 * shapes must be QKV H -> 3H, O H -> H, up H -> F, down F -> H (else RUDDER_ERR_SHAPE).  glue->out [M, ldout] receives
 * the block output.  Workspace: rudder_block_dit_workspace_bytes(args, M), 256-byte aligned.
 * rmsnorm, gelu and the additions are the bit-defined forms of rudder_rmsnorm, rudder_gelu and rudder_add below. */
typedef struct {
    const float* norm1_weight;   /* [H] fp32, 16-byte aligned */
    const float* norm2_weight;   /* [H] fp32, 16-byte aligned */
    float eps;                   /* >= 0 */
    uint16_t* out;               /* bf16 [M, ldout] */
    int64_t ldout;
} rudder_block_glue;
size_t rudder_block_dit_workspace_bytes(const rudder_block_args* args, int M);
rudder_status rudder_block_dit(const rudder_block_args* args, const rudder_block_glue* glue, int M, const rudder_segments* seg,
                               int step, void* workspace, size_t workspace_bytes, void* stream);

/* Measurement hook: rudder_block with a CUDA event between consecutive kernels.  ms (HOST [8])
 * receives the device time of each launch in order: prologue and GEMM of QKV, O, up, down.
 * Creates and destroys its events and SYNCHRONISES the stream before returning. */
rudder_status rudder_block_profile(const rudder_block_args* args, int M, const rudder_segments* seg, int step,
                                   void* workspace, size_t workspace_bytes, void* stream, float* ms);

/* rudder_block for callers whose activations live in HOST memory (pinned for asynchronous copies):
 * args->x[l] and args->y[l] are HOST pointers here (rows contiguous: ldx[l] >= K_l, ldy[l] >= N_l);
 * everything else is as in rudder_block.  Each input is copied to `staging`, the block runs, each
 * output is copied back, without synchronising: work queued on `stream` before the call precedes it,
 * work queued after the call follows the last copy.  Inside, uploads and downloads run on two
 * library-owned streams (created on first use, one pair per device) so that they overlap each other
 * and the kernels; concurrent host threads must therefore not call this on the same device.
 * staging: device memory of at least rudder_block_host_staging_bytes(args, M) bytes, 256-byte
 * aligned. */
size_t rudder_block_host_staging_bytes(const rudder_block_args* args, int M);
rudder_status rudder_block_host(const rudder_block_args* args, int M, const rudder_segments* seg, int step,
                                void* staging, size_t staging_bytes, void* workspace, size_t workspace_bytes,
                                void* stream);

/* ---------------------------------------------------------------------------------------------
 * Parity hooks: the production kernels, with their intermediate results written in canonical form.
 */
/* First kernel alone (Section 4.4): codes int8 [M, K] one code per byte (integer schemes) or
 * uint8 [M, K/2] packed E2M1, low nibble = even k (NVFP4); block_scales UE4M3 [M, K/16] (NVFP4
 * only, else NULL); row_scale fp32 [M]. */
rudder_status rudder_quantize_activations(const rudder_weight* w, const uint16_t* X, int64_t ldx, int M,
                                          const rudder_segments* seg, int step,
                                          const rudder_scale_table* tab, void* codes,
                                          uint8_t* block_scales, float* row_scale, void* stream);
/* The fused pass of a chained down projection alone (see rudder_block): X is the tensor BEFORE the GELU; the codes
 * (int8 [M, K], one per byte) and row scales are those of bf16(gelu(X)).  Static range and integer schemes only
 * (RUDDER_ERR_UNSUPPORTED otherwise). */
rudder_status rudder_gelu_quantize_activations(const rudder_weight* w, const uint16_t* X, int64_t ldx, int M,
                                               const rudder_segments* seg, int step, const rudder_scale_table* tab,
                                               void* codes, float* row_scale, void* stream);
/* rudder_linear that also writes the INT32 group accumulators C^(g) (Section 4.4: "accumulates
 * C = Q_X Q_W in INT32") of rows [row0, row0+rows) x columns [col0, col0+cols) into
 * acc int32 [K/group][rows][cols].  Integer schemes only.  row0 % 128 == 0 and col0 % 64 == 0. */
rudder_status rudder_linear_dump_acc(const rudder_weight* w, const uint16_t* X, int64_t ldx, int M,
                                     const rudder_segments* seg, int step, const rudder_scale_table* tab,
                                     const float* bias, uint16_t* Y, int64_t ldy,
                                     void* workspace, size_t workspace_bytes, void* stream,
                                     int row0, int rows, int col0, int cols, int32_t* acc);

/* BF16 GELU, elementwise, Y = bf16(gelu(X)): the glue of a chained block (the paper keeps GELU in BF16,
 * Appendix "Quantization"; which GELU is not stated).  Reading: the tanh form
 *   gelu(x) = x/2 (1 + tanh(0.7978845608 (x + 0.044715 x^3)))
 * with tanh u replaced by its [7/6] Pade approximant
 *   u (135135 + 17325 u^2 + 378 u^4 + u^6) / (135135 + 62370 u^2 + 3150 u^4 + 28 u^6)   for |u| < 5, +-1 beyond,
 * evaluated in fp32 by Horner's rule from the highest power, every add, multiply and the one divide
 * rounded to nearest on its own (no fused multiply-add): the result is defined bit for bit.
 * X, Y bf16 [M, ld]; N % 8 == 0; 16-byte aligned pointers, leading dimensions multiples of 8. */
rudder_status rudder_gelu(const uint16_t* X, int64_t ldx, int M, int N, uint16_t* Y, int64_t ldy, void* stream);

/* BF16 RMS normalisation of every row with a weight per channel (which normalisation the paper's models use is not
 * stated; reading: RMSNorm): Y = bf16((x * r) * weight), r = 1 / sqrt(mean(x^2) + eps).  Defined bit for bit: fp32, one
 * warp per row, lane l adds x * x (product and sum rounded separately) of the 8-value pieces l, l + 32, ... in order; the
 * 32 partial sums are combined by the exchange l ^ 16, 8, 4, 2, 1; mean = sum / N, r by IEEE division and square root.
 * X, Y bf16 [M, ld], weight fp32 [N]; N % 8 == 0; 16-byte aligned pointers, leading dimensions multiples of 8. */
rudder_status rudder_rmsnorm(const uint16_t* X, int64_t ldx, int M, int N, const float* weight, float eps, uint16_t* Y, int64_t ldy,
                             void* stream);
/* BF16 residual addition, elementwise: Y = bf16(A + B), one fp32 addition.  Same shape and alignment rules. */
rudder_status rudder_add(const uint16_t* A, int64_t lda, const uint16_t* B, int64_t ldb, int M, int N, uint16_t* Y, int64_t ldy,
                         void* stream);

/* Reads and clears the device status word (SYNCHRONISES the device).  *last (HOST) receives
 * RUDDER_OK or RUDDER_ERR_TIMEOUT; *where (HOST, may be NULL) a code naming the wait that gave up. */
rudder_status rudder_device_status(int* last, int* where);

/* Self-test of the bounded-wait path (no counterpart in the paper): launches ONE warp that waits, for at
 * most limit_cycles SM clocks (1e3 .. 1e8), on a barrier that nothing signals -- no copy, no tensor memory,
 * nothing in flight -- gives up, records RUDDER_ERR_TIMEOUT with the wait code 901 in the device status word
 * and returns normally.  The context stays usable; rudder_device_status then reports and clears the word. */
rudder_status rudder_selftest_wait_timeout(long long limit_cycles, void* stream);

const char* rudder_status_string(rudder_status s);

#ifdef __cplusplus
}
#endif
#endif /* RUDDER_H */
