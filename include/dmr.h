/*
 * libdmr: low-bit and step-routed decoder linear layers for Dynamic Mixed-Precision Routing,
 * written for NVIDIA B200 (sm_100a).  Plain C ABI: pointers and sizes only.
 *
 * The operations follow the paper's problem statement:
 *   - Sec. 3 (Problem Formulation): a set of LLMs derived from one base model under different
 *     numerical precisions; a routing index r_t chosen per step (Eq. 1) selects which precision
 *     serves that step.
 *   - Sec. 5 "Experimental Models and Precision" and App. "Quantization Detail": the
 *     low-precision model is W4A16 weight-only quantization of every decoder Linear layer
 *     (activations stay 16 bit), with a W3A16 group-128 variant as the most aggressive cell; the
 *     high-precision reference is bf16.
 *   - Sec. 4.2 "KL-to-Classification Mapping": label 1 means the step needs high precision.
 * The paper fixes no quantization arithmetic; the scheme implemented here is round-to-nearest
 * asymmetric min/max quantization with an integer zero point and a bf16 scale per group of
 * consecutive input features (see dmr_quantize).
 *
 * Conventions
 *   W  [N][K] bf16, row-major (N = out features, K = in features, like a Linear weight)
 *   X  [M][K] bf16, row-major (M = tokens, or concurrent agent steps)
 *   Y  [M][N] bf16 or fp32, row-major
 *   qweight [N][K*bits/32] uint32.  bits = 4: code k of a row is in word k/8, bits 4*(k%8)..+3.
 *                                   bits = 8: code k is in word k/4, bits 8*(k%4)..+7.
 *                                   bits = 3: every 32 codes take three words.  Code i < 30 of the block is
 *                                   in word i/10, at bits 3*(i%10)..+2 for i%10 < 5 and at bits
 *                                   16+3*(i%10-5)..+2 otherwise (five codes per half-word; bits 15 and 31
 *                                   stay free); bit b of code 30 is bit 15 of word b, bit b of code 31 is
 *                                   bit 31 of word b.  (The paper serves its 3-bit checkpoint expanded to
 *                                   fp16 and gives no packed layout; this one is the library's own: a
 *                                   half-word holds five codes that one mask turns into bf16 values.)
 *                                   Codes are unsigned, 0 .. 2^bits-1.
 *   scales  [N][G] bf16, zeros [N][G] uint8, G = K / g, g = group_size (0 means g = K).
 *   Dequantized weight: scale * (code - zero).
 *
 * Unless a parameter says "host", every data pointer is a DEVICE pointer owned by the caller.
 * The library allocates no device memory.  `stream` is a cudaStream_t passed as void*; all work
 * is enqueued on it and no call synchronises the host.  Argument errors are reported before
 * anything is launched.  Pointers must be 16-byte aligned.
 *
 * Threads.  Every entry point may be called from several host threads at once as long as calls that can
 * overlap on the GPU use different workspaces (and outputs).  The library's own host state - a cache of TMA
 * tensor maps keyed by address and shape, the per-kernel set-up flags, the launch counter - is guarded
 * inside; dmr_routed_linear calls of one process take turns while they enqueue (they share one helper stream
 * per device), which costs host time only.  dmr_last_cuda_error reports the last failure of any thread.
 */
#ifndef DMR_H_
#define DMR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DMR_OK = 0,
    DMR_ERR_INVALID_ARG = 1, /* null pointer, negative size, K not a multiple of the group ... */
    DMR_ERR_UNSUPPORTED = 2, /* a format or shape the library has no kernel for */
    DMR_ERR_ALIGNMENT = 3,   /* a pointer is not 16-byte aligned */
    DMR_ERR_WORKSPACE = 4,   /* workspace is NULL or smaller than dmr_workspace_bytes() */
    DMR_ERR_NONFINITE = 5,   /* written to dev_status by dmr_quantize: NaN/Inf weight seen */
    DMR_ERR_TIMEOUT = 6,     /* written to the workspace status word: a bounded wait ran out */
    DMR_ERR_CUDA = 7         /* a CUDA call failed; see dmr_last_cuda_error() */
} dmr_status_t;

typedef struct {
    int32_t bits;       /* 3, 4 or 8 */
    int32_t group_size; /* 64, 128, ... (multiple of 32, divides K), or 0 = one group per row */
} dmr_qformat_t;

typedef enum { DMR_OUT_BF16 = 0, DMR_OUT_F32 = 1 } dmr_out_t;

typedef enum {
    DMR_OP_LOWBIT_LINEAR = 0,
    DMR_OP_DENSE_LINEAR = 1,
    DMR_OP_ROUTED_LINEAR = 2
} dmr_op_t;

/* Sizes of the quantized tensors in bytes (0 if the format is invalid for K). */
size_t dmr_qweight_bytes(int N, int K, dmr_qformat_t f);
size_t dmr_scales_bytes(int N, int K, dmr_qformat_t f);
size_t dmr_zeros_bytes(int N, int K, dmr_qformat_t f);

/* Scratch bytes `op` needs for these sizes (split-K partial sums, routed row lists and
 * compacted activations, decode counters, a status word).  Always a multiple of 256; never 0.
 * The workspace must be zero-filled once before its first use; every call leaves the words that
 * have to be zero (counters, status) zero again, so it can be reused without clearing.  Calls
 * that may overlap on the GPU need separate workspaces. */
size_t dmr_workspace_bytes(dmr_op_t op, int M, int N, int K, dmr_qformat_t f);

/*
 * Quantize and pack bf16 weights (the low-precision model of Sec. 5 / App. "Quantization
 * Detail": weight-only, 16-bit activations).  Per row n and group j of g consecutive k, in
 * binary64, with qmax = 2^bits - 1:
 *   lo = min(0, min w), hi = max(0, max w);  s = nearest bf16 to (hi - lo) / qmax (ties to
 *   even; 1.0 for an all-zero group; raised to 2^-126 if it would be zero or subnormal);
 *   zero = clamp(rint(-lo / s), 0, qmax);  code_k = clamp(rint(w_k / s) + zero, 0, qmax).
 * Outputs: qweight, scales, zeros as laid out above.  dev_status: one int32 on the device,
 * set to DMR_ERR_NONFINITE if any weight is NaN or Inf (outputs are then unspecified) and
 * left untouched otherwise; the caller zeroes it beforehand.  May be NULL.
 * Requires K % g == 0, g % 32 == 0, K % 32 == 0.
 */
dmr_status_t dmr_quantize(const void *W_bf16, int N, int K, dmr_qformat_t f, void *qweight,
                          void *scales, void *zeros, int32_t *dev_status, void *stream);

/* Test utility: W_out[n][k] = scale * (code - zero), as fp32 (exact) or bf16 (nearest): the weights the
 * low-precision model of Sec. 5 / App. "Quantization Detail" computes with, written out. */
dmr_status_t dmr_dequantize(const void *qweight, const void *scales, const void *zeros, int N,
                            int K, dmr_qformat_t f, void *W_out, dmr_out_t out, void *stream);

/*
 * Low-precision linear layer (the W4A16 model's Linear, Sec. 5; also 8-bit and 3-bit codes): Y = X . dequant(Wq)^T
 * with fp32 accumulation.  Up to 32 rows run the bandwidth-bound decode kernels, larger M the tensor-core
 * kernels (3-bit codes: the persistent tensor-core kernel where it applies, otherwise the decode kernel, 16 rows per launch).  The decode kernels start fetching qweight, scales and zeros before the preceding kernel
 * of `stream` has finished (programmatic dependent launch): these three must be complete when the
 * call is enqueued, or be written by kernels that do not release their dependents early (dmr_quantize
 * and every ordinary kernel launch qualify).  X may be produced by the preceding kernel.
 * M = 0 is a no-op.  workspace: dmr_workspace_bytes(DMR_OP_LOWBIT_LINEAR, ...) bytes.
 */
dmr_status_t dmr_lowbit_linear(const void *X_bf16, int M, const void *qweight, const void *scales,
                               const void *zeros, int N, int K, dmr_qformat_t f, void *Y,
                               dmr_out_t out, void *workspace, size_t workspace_bytes,
                               void *stream);

/* High-precision linear layer (the bf16 reference model, Sec. 5): Y = X . W^T, fp32 accumulation. */
dmr_status_t dmr_dense_linear(const void *X_bf16, int M, const void *W_bf16, int N, int K, void *Y,
                              dmr_out_t out, void *workspace, size_t workspace_bytes, void *stream);

/*
 * Step-routed linear layer (Sec. 3, Eq. 1: the router picks a precision per step; Sec. 4.2:
 * label 1 = high precision).  mask [M] uint8 on the device: rows with mask != 0 are multiplied
 * with the bf16 weights W, the others with the low-bit weights; every row's result is written
 * at its own index m, so Y is in step order.  The mask is read on the device only.  Row m equals,
 * bit for bit, row m of dmr_dense_linear (mask != 0) or dmr_lowbit_linear (mask == 0) called
 * on the same M rows.  The two halves run concurrently: the library forks a helper stream after the
 * partition and joins it back into `stream` before returning (also under stream capture).  The
 * helper stream and its two events are created by the first routed call on a device; make that
 * first call outside any capture.
 */
dmr_status_t dmr_routed_linear(const void *X_bf16, int M, const uint8_t *mask, const void *W_bf16,
                               const void *qweight, const void *scales, const void *zeros, int N,
                               int K, dmr_qformat_t f, void *Y, dmr_out_t out, void *workspace,
                               size_t workspace_bytes, void *stream);

/*
 * Stable partition of step indices by mask (the split that dmr_routed_linear performs first): the per-step
 * routing index r_t of Sec. 3, Eq. 1, turned into the two lists of steps each precision serves; mask != 0
 * marks the steps whose router score reached the threshold of Sec. 4.2 "Inference-time calibration".
 * idx_high / idx_low: int32 [M] each; counts: int32 [2] = {n_high, n_low}.  All on the device.
 */
dmr_status_t dmr_route_partition(const uint8_t *mask, int M, int32_t *idx_high, int32_t *idx_low,
                                 int32_t *counts, void *stream);

/*
 * dmr_lowbit_linear for callers whose activations live in host memory: X_host [M][K] bf16 and
 * Y_host [M][N] are HOST pointers (pinned memory makes the copies asynchronous); the weights stay
 * on the device.  The call copies X to the device, runs the layer and copies Y back, all on
 * `stream`, and returns without synchronising.  staging: device scratch of
 * dmr_host_staging_bytes(M, N, K, out) bytes.
 */
size_t dmr_host_staging_bytes(int M, int N, int K, dmr_out_t out);
dmr_status_t dmr_lowbit_linear_host(const void *X_host, int M, const void *qweight,
                                    const void *scales, const void *zeros, int N, int K,
                                    dmr_qformat_t f, void *Y_host, dmr_out_t out, void *staging,
                                    size_t staging_bytes, void *workspace, size_t workspace_bytes,
                                    void *stream);

/*
 * No counterpart in the paper: a variant of dmr_lowbit_linear (M <= 16, the decode kernel) for
 * callers that cannot allocate device memory when they call - for example a serving loop that
 * gave all free memory to its cache pool at start-up, or code running inside another program's
 * step that must not touch its allocator (cudaMalloc can also stall the whole device).  It takes
 * no workspace: the kernel's scratch (counters, partial sums, a status word; about 8.5 MB) is a
 * fixed array inside the library, which every GPU that loads the library holds until exit.
 *   - Limits: 1 <= M <= 16, N <= dmr_noalloc_max_n() (65536), formats the decode kernel takes
 *     (4-bit with group 64 or a multiple of 128, 8-bit with a multiple of 64); anything else
 *     returns DMR_ERR_UNSUPPORTED and launches nothing.  X, qweight, scales, zeros and Y are the
 *     caller's device buffers exactly as for dmr_lowbit_linear.  It always runs the shared-memory-ring
 *     streaming kernel, so its result agrees with dmr_lowbit_linear's up to the order of the fp32 sums
 *     (a few 1e-6 of the largest output), not bit for bit.
 *   - The first call on each device looks up the array's device address (no allocation); make
 *     that first call with the device current and before any stream capture begins.
 *   - The call allocates and frees nothing.  It clears the status word itself; all calls on one
 *     device share the one array, so two calls that may run on the GPU at the same time (two
 *     streams, two threads) race - serialise them or use dmr_lowbit_linear with workspaces.
 */
int dmr_noalloc_max_n(void);
dmr_status_t dmr_lowbit_linear_noalloc(const void *X_bf16, int M, const void *qweight, const void *scales,
                                       const void *zeros, int N, int K, dmr_qformat_t f, void *Y,
                                       dmr_out_t out, void *stream);

/*
 * Step-wise KL divergence between the high- and the low-precision model's action distributions,
 * the signal the KL-ST router is trained on (Sec. "KL-ST Stage"; App. on search and click steps:
 * KL_t = mean over the action tokens i of step t of KL(pi_high(x_i) || pi_low(x_i))).
 *   logits_high, logits_low : device, [T][V] row-major, bf16 (dtype = DMR_OUT_BF16) or fp32
 *                             (DMR_OUT_F32); row i holds the logits both models give for action
 *                             token i.  16-byte aligned.  Read once, not modified.
 *   step_offsets            : device, int32 [S + 1], non-decreasing, within [0, T]: step s owns the
 *                             tokens [step_offsets[s], step_offsets[s + 1]).  May be NULL when S = 0.
 *   kl_token                : device, fp32 [T], written: KL(softmax(high_i) || softmax(low_i)) in nats.
 *   kl_step                 : device, fp32 [S], written: the mean of kl_token over the step's tokens
 *                             (added in token order), 0 for a step without tokens.
 * fp32 arithmetic, one pass over the logits; a vocabulary entry with probability 0 under the
 * high-precision model (logit -inf) contributes nothing.  No workspace, no allocation.
 * Errors: DMR_ERR_INVALID_ARG (null pointer, T < 0, V < 1, S < 0, bad dtype), DMR_ERR_ALIGNMENT,
 * DMR_ERR_CUDA.  T = 0 writes only kl_step (zeros).  The caller owns all buffers.
 */
dmr_status_t dmr_stepwise_kl(const void *logits_high, const void *logits_low, dmr_out_t dtype, int T,
                             int V, const int32_t *step_offsets, int S, float *kl_token, float *kl_step,
                             void *stream);

/*
 * Inference-time calibration of the router (Sec. 4.2 "Inference-time calibration"): for a high-precision budget
 * rho the threshold is tau(rho) = Quantile(D_cal, 1 - rho) over the router's scores on a calibration pool (the
 * paper uses rho in {0.20, 0.40, 0.70}), and a step goes to the high-precision model when its score p_t >= tau.
 *   dmr_router_calibrate: cal_scores device fp32 [n], finite, 1 <= n <= 65536 (more: DMR_ERR_UNSUPPORTED);
 *       0 <= rho <= 1; tau: device, THREE doubles, 16-byte aligned - tau[0] receives the threshold, tau[1..2] are
 *       scratch.  Quantile rule (the paper names none): linear interpolation between order statistics,
 *       x_(lo) + (h - lo)(x_(lo+1) - x_(lo)) with h = (n - 1)(1 - rho), lo = floor(h), in binary64.
 *   dmr_router_mask: scores device fp32 [M] -> mask device uint8 [M], mask[m] = (scores[m] >= tau[0]) ? 1 : 0, the
 *       mask dmr_routed_linear takes (1 = high precision).  tau is read on the device: no host round trip between
 *       calibration, masking and the routed layer.  M = 0 is a no-op.
 * Errors: DMR_ERR_INVALID_ARG (null pointer, n < 1, M < 0, rho outside [0, 1]), DMR_ERR_ALIGNMENT, DMR_ERR_CUDA.
 */
dmr_status_t dmr_router_calibrate(const float *cal_scores, int n, double rho, double *tau, void *stream);
dmr_status_t dmr_router_mask(const float *scores, int M, const double *tau, uint8_t *mask, void *stream);

/*
 * Forward pass of the step-level router (Sec. 4.1 "Router Architecture"): the sequence X_t = [z_task, z_1, ..., z_t] of
 * task and step embeddings plus learned positional embeddings P_t goes through a masked Transformer encoder,
 * H_t = TransformerEnc(X_t + P_t, m_t); the encoder's output at the last valid step, h_t*, gives the distribution over
 * the precision choices, Softmax(W h_t*).  The paper fixes neither sizes, normalisation placement nor activation; the
 * layer implemented is the original Transformer's encoder layer: x <- LN(x + MHA(x)), x <- LN(x + W2 relu(W1 x + b1) + b2),
 * padded steps never attended to, no causal mask, LN eps 1e-5.  fp32 arithmetic.
 *   cfg: d (model width: multiple of 16, 16..1024), heads (divides d), ffn (multiple of 16), layers (1..64),
 *        l_max (positions, 1..128), classes (precision choices, 1..32).
 *   params: device fp32, dmr_router_param_floats(cfg) values, 16-byte aligned, in this order:
 *        pos [l_max][d];  per layer: wqkv [3d][d] (rows: queries, keys, values), bqkv [3d], wo [d][d], bo [d],
 *        ln1_g [d], ln1_b [d], w1 [ffn][d], b1 [ffn], w2 [d][ffn], b2 [d], ln2_g [d], ln2_b [d];  wc [classes][d], bc [classes].
 *   Z: device fp32 [B][L][d] (embeddings from the frozen encoder; L <= l_max; truncating a longer trajectory is the
 *        caller's choice).  lengths: device int32 [B], valid entries per sequence, valid steps first, 1 <= lengths[b] <= L
 *        (values outside are clamped into that range).  Entries of Z behind a sequence's length are ignored.
 *   probs: device fp32 [B][classes].  scores: NULL, or device fp32 [B] that receives probs[b][score_class] - the
 *        vector dmr_router_calibrate and dmr_router_mask take (score_class = the high-precision choice).
 *   workspace: dmr_router_workspace_bytes(cfg, B, L) bytes, 16-byte aligned, no initial contents required.
 * B = 0 is a no-op.  Errors: DMR_ERR_INVALID_ARG (sizes, NULL), DMR_ERR_ALIGNMENT, DMR_ERR_WORKSPACE.
 */
typedef struct {
    int32_t d, heads, ffn, layers, l_max, classes;
} dmr_router_cfg_t;
size_t dmr_router_param_floats(dmr_router_cfg_t cfg);               /* 0 if cfg is invalid */
size_t dmr_router_workspace_bytes(dmr_router_cfg_t cfg, int B, int L); /* 0 if cfg, B or L is invalid */
dmr_status_t dmr_router_forward(const float *params, dmr_router_cfg_t cfg, const float *Z, const int32_t *lengths, int B,
                                int L, float *probs, float *scores, int score_class, void *workspace,
                                size_t workspace_bytes, void *stream);

/*
 * Self-test of the bounded waits (no counterpart in the paper).  Every wait inside the kernels gives up after a
 * fixed number of polls, writes DMR_ERR_TIMEOUT to the workspace's status word and lets the kernel finish, so a
 * copy that never lands cannot hang the GPU.  This call launches one warp that waits - with the limit lowered
 * to a thousand polls - on a barrier nothing ever arrives at.  Afterwards dmr_workspace_status(workspace)
 * returns DMR_ERR_TIMEOUT and the second int32 of the workspace holds 2 (the kernel ran to its end).  The
 * caller clears the first 256 bytes of the workspace before using it for other calls again.
 * workspace: at least 256 bytes, zero-filled.
 */
dmr_status_t dmr_selftest_wait_timeout(void *workspace, size_t workspace_bytes, void *stream);

/* Reads the status word a previous call may have set in `workspace` (DMR_OK or DMR_ERR_TIMEOUT).
 * Synchronises `stream`. */
dmr_status_t dmr_workspace_status(const void *workspace, void *stream);

/*
 * Writes a one-line description of the kernel family and launch shape that dmr_lowbit_linear
 * (op = DMR_OP_LOWBIT_LINEAR) or dmr_dense_linear (DMR_OP_DENSE_LINEAR; f is ignored) would use for these sizes
 * on the current device, e.g. "prefill bits=4 bn=256 tiles=3072 ctas=148".  Launches nothing.  Returns the length
 * snprintf reports, or -1 for invalid arguments.  For tests and benchmarks that must know which kernel they ran.
 */
int dmr_describe_dispatch(dmr_op_t op, int M, int N, int K, dmr_qformat_t f, char *buf, size_t buf_bytes);

const char *dmr_status_string(dmr_status_t s);
int dmr_last_cuda_error(void);

/* Number of kernels this library has launched in this process (for launch accounting). */
uint64_t dmr_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* DMR_H_ */
